#!/usr/bin/env python
"""Long lock-step run of one workload: the CUDA path against the CPU oracle, step by step.

Test infrastructure (it imports the oracle); not collected by pytest.  For every step the
accepted lengths, next tokens, rescue masks and rejection lists must be identical; the
diagnostics (t*, m, counts exact; s, lse, score, p_d, p_t within 1e-5) are compared on the
first 100 steps and every 100th after; the memory's (pair, count) set, n_keys and n_dropped
are compared at every checkpoint and at the end.  Prints one JSON line per (workload, tau).

    python tests/lockstep_run.py --workload ocm_contention --steps 20000 --checkpoint 10000
"""

import argparse
import json
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import test_gpu_parity as T                                     # noqa: E402
from oracle import csd_oracle as ORACLE                          # noqa: E402
from paper_2604_13634_b200 import Ocm, StepBuffers, csd_step     # noqa: E402
from synth_inputs import WORKLOADS, Synth         # noqa: E402


OVERLAP = False
_PINNED = {}


def _bits_through_pinned_memory(z: torch.Tensor):
    """Same result as synth_inputs.logits_bits_numpy, but the device-to-host copy lands in a pinned buffer
    that is kept between steps (several times faster for the 100 MB+ steps of the long runs)."""
    z = z.detach().contiguous()
    key = (tuple(z.shape), z.dtype)
    if key not in _PINNED:
        _PINNED.clear()
        _PINNED[key] = torch.empty(z.shape, dtype=z.dtype).pin_memory()
    host = _PINNED[key]
    host.copy_(z, non_blocking=False)
    if z.dtype == torch.bfloat16:
        return host.view(torch.int16).numpy().view("uint16"), True
    return host.numpy(), False


T.logits_bits_numpy = _bits_through_pinned_memory


def compare_memory(ocm, mem, dropped_before=0):
    """Stored pairs, counts, number of keys and of dropped occurrences (a continued run's library
    object counts its drops from the leg's start)."""
    d, t, c = ocm.export()
    rd, rt, rc = mem.export()
    assert np.array_equal(d.numpy(), rd) and np.array_equal(t.numpy(), rt), "stored pairs differ"
    assert np.array_equal(c.numpy(), rc), "counts differ"
    st = ocm.stats()
    assert st["n_keys"] == mem.n_keys and st["n_dropped"] + dropped_before == mem.n_dropped
    return st


def save_state(path, mem, next_step, totals):
    d, t, c = mem.export()
    np.savez(path, d=d, t=t, c=c, n_dropped=mem.n_dropped, next_step=next_step, totals=np.asarray(totals, dtype=np.int64))


def load_state(path, ocm, mem):
    """Continue a run: the oracle's memory comes from the file, the library's is loaded with the same
    triples (the previous leg ended with the two compared equal)."""
    st = np.load(path)
    mem.table = {(int(a), int(b)): int(c) for a, b, c in zip(st["d"], st["t"], st["c"])}
    mem.n_dropped = int(st["n_dropped"])
    if len(st["d"]):
        dev = ocm.device
        ocm.import_(torch.tensor(st["d"], dtype=torch.int32, device=dev), torch.tensor(st["t"], dtype=torch.int32, device=dev),
                    torch.tensor(st["c"], dtype=torch.int64, device=dev).to(torch.int32))
    return int(st["next_step"]), [int(x) for x in st["totals"]]


def run(wl, tau, steps, checkpoint, prewarm_steps, seed=0, first_step=None, load=None, save=None):
    syn = Synth(wl, seed, "cuda")
    ocm = Ocm(wl.ocm_slots, wl.lam)
    mem = ORACLE.OCM(wl.ocm_slots, wl.lam)
    kind, n = wl.prewarm
    resumed = None
    if load:
        resumed = load_state(load, ocm, mem)
        kind = "none"
    if kind == "pairs":
        pd, pt = syn.prewarm_pairs(n)
        ocm.update(pd, pt)
        mem.update(zip(pd.cpu().tolist(), pt.cpu().tolist()))
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
    first = 0
    if kind == "steps":
        # pre-warming steps are ordinary steps of the same stream, checked like the others
        first = -min(prewarm_steps, n)
    t0 = time.time()
    near = acc = resc = checked_diag = 0
    dropped_before = 0
    if resumed:
        first, (near, acc, resc, checked_diag) = resumed
        dropped_before = mem.n_dropped          # the library counts drops from this leg's start
    if first_step is not None and not resumed:
        first = first_step
    for s in range(first, steps):
        z, d = syn.step(s + 10 ** 6 if s < 0 else s)
        csd_step(z, d, ocm, tau, buf)
        ref = T.oracle_step(z, d, mem, tau)
        sample = (s < 100) or (s % 100 == 0)
        near += T.compare(buf, ref, check_diag=sample)
        checked_diag += int(sample)
        if s >= 0:
            acc += int(ref["accept_len"].sum())
            resc += int(ref["rescued_mask"].sum())
        if checkpoint and s >= 0 and (s + 1) % checkpoint == 0:
            compare_memory(ocm, mem, dropped_before)
    st = compare_memory(ocm, mem, dropped_before)
    assert st["flags"] == 0, st
    if save:
        save_state(save, mem, steps, (near, acc, resc, checked_diag))
    out = dict(workload=wl.name, tau=tau, steps=steps, prewarm_steps=-first, B=wl.B, K=wl.K, V=wl.V, dtype=wl.dtype,
               first_step_of_this_leg=first, accepted=acc, rescued=resc,
               acceptance_rate=acc / (steps * wl.B * wl.K), near_ties=near,
               diag_steps_checked=checked_diag, n_keys=st["n_keys"], n_dropped=st["n_dropped"],
               checkpoints=(steps // checkpoint if checkpoint else 0), seconds=round(time.time() - t0, 1),
               overlap_launch_shape=bool(OVERLAP), verdict="identical")
    ocm.close()
    return out


def run_sampled(wl, tau, steps, T_, lam, seed=0):
    """The stochastic step (Algorithm 1 at temperature T_) in lock-step with its oracle.  A batch row
    whose result hangs on a near-tie the oracle flags is counted as excused and the memories are
    re-synchronised; any other difference raises."""
    import test_gpu_sampled_parity as S
    from paper_2604_13634_b200 import SampledBuffers, csd_step_sampled
    syn = Synth(wl, seed, "cuda")
    ocm, mem = Ocm(wl.ocm_slots, lam), S.ORACLE.OCM(wl.ocm_slots, lam)
    buf = SampledBuffers(wl.B, wl.K, wl.V, wl.torch_dtype)
    t0 = time.time()
    excused = passed = resc = acc = flagged = 0
    for s in range(steps):
        z, y, d, r = syn.step_sampled(s)
        csd_step_sampled(z, y, d, r, 7919 * seed + s, T_, ocm, tau, buf)
        ref = S.oracle_sampled(z, y, d, r, 7919 * seed + s, T_, mem, tau)
        e = S.compare(buf, ref)
        excused += e
        if e:
            S.resync(ocm, mem)
        flagged += int(ref["near_accept"].sum()) + int(ref["unclear_draw"].sum())
        passed += int(ref["accepted"].sum())
        resc += int(ref["rescued_mask"].sum())
        acc += int(ref["accept_len"].sum())
        if (s + 1) % 100 == 0:
            S.compare_memory(ocm, mem)
    st = S.compare_memory(ocm, mem)
    assert st["flags"] == 0, st
    out = dict(workload=wl.name, mode="stochastic", temperature=T_, tau=tau, lam=lam, steps=steps, B=wl.B, K=wl.K, V=wl.V,
               dtype=wl.dtype, passed_acceptance_test=passed, rescued=resc, accepted=acc,
               acceptance_rate=acc / (steps * wl.B * wl.K), near_ties_flagged_by_oracle=flagged,
               batch_rows_excused=excused, n_keys=st["n_keys"], seconds=round(time.time() - t0, 1),
               verdict="identical apart from the excused rows")
    ocm.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", required=True)
    ap.add_argument("--steps", type=int, default=0, help="0 = the workload's own step count")
    ap.add_argument("--checkpoint", type=int, default=0)
    ap.add_argument("--prewarm-steps", type=int, default=10 ** 9, help="cap on step-type pre-warming")
    ap.add_argument("--taus", default="")
    ap.add_argument("--load", default="", help="continue from a state file written by --save")
    ap.add_argument("--save", default="", help="write the memory and the running totals here at the end")
    ap.add_argument("--overlap", action="store_true",
                    help="the launch shape the benchmark times (csd_set_overlap: one block per SM and launch)")
    ap.add_argument("--sampled", type=float, default=0.0,
                    help="run the stochastic step at this temperature instead of the greedy one")
    ap.add_argument("--lam", type=int, default=2, help="frequency threshold of the --sampled run")
    args = ap.parse_args()
    if args.sampled > 0:
        wl = WORKLOADS[args.workload]
        for tau in ([float(x) for x in args.taus.split(",")] if args.taus else list(wl.taus)):
            print(json.dumps(run_sampled(wl, tau, args.steps or wl.steps, args.sampled, args.lam)), flush=True)
        return
    if args.overlap:
        from paper_2604_13634_b200 import csd_set_overlap
        global OVERLAP
        OVERLAP = True
        csd_set_overlap(True)
    wl = WORKLOADS[args.workload]
    taus = [float(x) for x in args.taus.split(",")] if args.taus else list(wl.taus)
    for tau in taus:
        res = run(wl, tau, args.steps or wl.steps, args.checkpoint or wl.checkpoint_every, args.prewarm_steps,
                  load=args.load or None, save=args.save or None)
        print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
