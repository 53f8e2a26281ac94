"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bar: accepted lengths, next tokens, rescue masks, rejection lists, arg-max indices,
maxima, gathered logits, look-up counts and the memory's (pair, count) set bit-exact;
s, lse, score, p_d, p_t within 1e-5 relative (fp32 arithmetic against the fp64 oracle).
Positions whose score lies within 1e-5 of tau are counted and reported; because the
gate is decided exactly on both sides they are expected to agree as well.
"""

import dataclasses
import os

import numpy as np
import pytest
import torch

from oracle import csd_oracle as ORACLE
from oracle import row_stats_c
from paper_2604_13634_b200 import (CSD_BF16, CSD_F32, HostStep, Ocm, StepBuffers, csd_launch_shape, csd_set_tuning,
                                   csd_step, csd_verify)
from synth_inputs import WORKLOADS, Synth, logits_bits_numpy

pytestmark = pytest.mark.gpu

RTOL = 1e-5


class _Bf16Decoded:
    """bf16 bit patterns that decode on access: the oracle step only gathers single logits once the row
    statistics come from the C routine, so widening a 100 MB tensor every step would be wasted."""

    def __init__(self, bits):
        self.bits = bits
        self.shape = bits.shape

    def __getitem__(self, idx):
        return ORACLE.bf16_bits_to_f64(np.asarray(self.bits[idx])).reshape(np.shape(self.bits[idx]))


def _np_logits(z, lazy=False):
    arr, is_bits = logits_bits_numpy(z)
    if is_bits:
        return (_Bf16Decoded(arr) if lazy else ORACLE.bf16_bits_to_f64(arr).astype(np.float32)), arr, True
    return arr, arr, False


def oracle_step(z, draft, mem, tau, update=True, use_c=True):
    vals, raw, is_bits = _np_logits(z, lazy=use_c and z.is_contiguous())
    stats = None
    if use_c and z.is_contiguous():
        stats = row_stats_c.row_stats_batch(raw, is_bf16_bits=is_bits)
    d = draft.cpu().numpy()
    return ORACLE.step(vals, d, mem, tau, stats=stats) if update else ORACLE.verify(vals, d, mem, tau, stats=stats)


def assert_close(name, got, ref, rtol=RTOL, atol=1e-37):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    both_nan = np.isnan(got) & np.isnan(ref)
    bad = ~both_nan & ~(np.abs(got - ref) <= rtol * np.abs(ref) + atol)
    assert not bad.any(), f"{name}: {int(bad.sum())} entries beyond {rtol}: got {got[bad][:4]} ref {ref[bad][:4]}"


def compare(buf: StepBuffers, ref, check_diag=True):
    g = lambda t: t.cpu().numpy()
    for k in ("accept_len", "next_token", "rescued_mask"):
        assert np.array_equal(g(getattr(buf, k)), ref[k]), k
    assert np.array_equal(g(buf.rej_draft), ref["rej_draft"]), "rej_draft"
    assert np.array_equal(g(buf.rej_target), ref["rej_target"]), "rej_target"
    if check_diag and buf.diag is not None:
        dg = {k: g(v) for k, v in buf.diag.items()}
        assert np.array_equal(dg["t"], ref["t"]), "t"
        assert np.array_equal(dg["m"].astype(np.float64), ref["m"]), "m"
        assert np.array_equal(dg["cnt"].astype(np.int64) & 0xFFFFFFFF, ref["cnt"]), "cnt"
        zd_ref = ref["zd"]
        assert np.array_equal(np.isnan(dg["zd"]), np.isnan(zd_ref))
        ok = ~np.isnan(zd_ref)
        assert np.array_equal(dg["zd"][ok].astype(np.float64), zd_ref[ok]), "zd"
        assert_close("s", dg["s"], ref["s"])
        assert_close("lse", dg["lse"], ref["lse"])
        assert_close("score", dg["score"], ref["score"])
        assert_close("p_d", dg["p_d"], ref["p_d"])
        assert_close("p_t", dg["p_t"], ref["p_t"])
    return int(ref["near_tie"].sum())


def compare_memory(ocm: Ocm, mem: ORACLE.OCM):
    d, t, c = ocm.export()
    rd, rt, rc = mem.export()
    assert np.array_equal(d.numpy(), rd) and np.array_equal(t.numpy(), rt), "stored pairs differ"
    assert np.array_equal(c.numpy(), rc), "counts differ"
    st = ocm.stats()
    assert st["n_keys"] == mem.n_keys and st["n_dropped"] == mem.n_dropped
    return st


def lockstep(wl, steps, tau, lam=None, seed=0, diag=True, prewarm_pairs=0, first_step=0, check_every=0):
    lam = wl.lam if lam is None else lam
    syn = Synth(wl, seed, "cuda")
    ocm = Ocm(wl.ocm_slots, lam)
    mem = ORACLE.OCM(wl.ocm_slots, lam)
    if prewarm_pairs:
        pd, pt = syn.prewarm_pairs(prewarm_pairs)
        ocm.update(pd, pt)
        mem.update(zip(pd.cpu().tolist(), pt.cpu().tolist()))
        compare_memory(ocm, mem)
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=diag)
    near = 0
    tot = dict(acc=0, resc=0)
    for s in range(first_step, first_step + steps):
        z, d = syn.step(s)
        csd_step(z, d, ocm, tau, buf)
        ref = oracle_step(z, d, mem, tau)
        near += compare(buf, ref)
        tot["acc"] += int(ref["accept_len"].sum())
        tot["resc"] += int(ref["rescued_mask"].sum())
        if check_every and (s + 1) % check_every == 0:
            compare_memory(ocm, mem)
    st = compare_memory(ocm, mem)
    assert st["flags"] == 0
    assert st["steps"] == steps and st["positions"] == steps * wl.B * wl.K
    ocm.close()
    return tot, near, st


# ---------------------------------------------------------------------------------------
# element-wise parity on small shapes: several tiles, ragged tails, both dtypes, both paths
# ---------------------------------------------------------------------------------------
SHAPES = [
    (3, 4, 5000, torch.float32), (2, 5, 20000, torch.bfloat16), (1, 1, 1, torch.float32), (1, 1, 8, torch.bfloat16),
    (2, 3, 4099, torch.float32),            # V not a multiple of 4: element-wise path
    (2, 3, 4099, torch.bfloat16),
    (4, 32, 3000, torch.bfloat16),          # K at the limit
    (5, 2, 70001, torch.float32), (2, 2, 1024 * 33 + 8, torch.bfloat16), (1, 7, 262144, torch.float32),
]


def _random_inputs(B, K, V, dtype, seed, match_p=0.5):
    g = torch.Generator(device="cuda").manual_seed(seed)
    z = torch.randn(B, K + 1, V, generator=g, device="cuda") * 2
    top = torch.randint(0, V, (B, K + 1), generator=g, device="cuda")
    z.scatter_add_(2, top.unsqueeze(-1), torch.full((B, K + 1, 1), 5.0, device="cuda"))
    z = z.to(dtype)
    arg = z[:, :K].float().argmax(dim=2)
    rnd = torch.randint(0, V, (B, K), generator=g, device="cuda")
    near = (arg + torch.randint(0, 3, (B, K), generator=g, device="cuda")) % V
    pick = torch.rand(B, K, generator=g, device="cuda")
    draft = torch.where(pick < match_p, arg, torch.where(pick < match_p + 0.25, near, rnd)).to(torch.int32)
    return z.contiguous(), draft.contiguous()


@pytest.mark.parametrize("B,K,V,dtype", SHAPES)
def test_elementwise_parity_small(B, K, V, dtype):
    ocm = Ocm(1024, 1)
    mem = ORACLE.OCM(1024, 1)
    buf = StepBuffers(B, K, V, dtype, diag=True)
    for rep in range(4):
        z, d = _random_inputs(B, K, V, dtype, seed=100 + rep)
        if rep >= 2:
            d = _random_inputs(B, K, V, dtype, seed=100 + rep - 2)[1]     # revisit pairs: rescues happen
            z = _random_inputs(B, K, V, dtype, seed=100 + rep - 2)[0]
        csd_step(z, d, ocm, 1e-4, buf)
        compare(buf, oracle_step(z, d, mem, 1e-4, use_c=(rep % 2 == 0)))
    compare_memory(ocm, mem)
    ocm.close()


def test_strided_and_misaligned_views():
    B, K, V = 3, 4, 6000
    for dtype in (torch.float32, torch.bfloat16):
        big, d = _random_inputs(B, K, V + 24, dtype, seed=7)
        for view in (big[:, :, :V], big[:, :, 1:V + 1], big[:, :, 8:V + 8]):
            d = d % V
            ocm = Ocm(256, 0)
            mem = ORACLE.OCM(256, 0)
            buf = StepBuffers(B, K, V, dtype, diag=True)
            csd_step(view, d, ocm, 0.05, buf)
            ref = ORACLE.step(view.float().cpu().numpy(), d.cpu().numpy(), mem, 0.05)
            compare(buf, ref)
            compare_memory(ocm, mem)
            ocm.close()


def test_ties_infinities_and_constant_rows():
    B, K, V = 4, 3, 9000
    z = torch.zeros(B, K + 1, V, device="cuda", dtype=torch.bfloat16)
    z[0] = 1.5                                   # constant rows: arg-max 0
    z[1, :, 4000:] = 2.0                         # plateau: lowest index 4000
    z[1, 1, 8999] = 2.0
    z[2] = float("-inf")
    z[2, :, 77] = -3.0                           # single finite value
    z[2, 1, 5000] = -3.0                         # tie with 77: lowest wins
    z[3] = torch.randn(K + 1, V, device="cuda").to(torch.bfloat16)      # real bf16 ties are likely
    d = torch.tensor([[0, 5, 0], [4000, 8999, 3], [77, 5000, 78], [1, 2, 3]], dtype=torch.int32, device="cuda")
    ocm = Ocm(256, 0)
    mem = ORACLE.OCM(256, 0)
    buf = StepBuffers(B, K, V, torch.bfloat16, diag=True)
    csd_step(z, d, ocm, 0.9, buf)
    ref = oracle_step(z, d, mem, 0.9)
    compare(buf, ref)
    assert buf.diag["t"][0].tolist() == [0, 0, 0, 0] and buf.diag["t"][1, 0].item() == 4000
    assert buf.accept_len.tolist()[:3] == [3, 2, 2]       # score 1 at a tie passes tau = 0.9
    compare_memory(ocm, mem)
    assert ocm.stats()["flags"] == 0
    ocm.close()


def test_bad_inputs_flag_and_never_rescue():
    B, K, V = 2, 4, 5000
    z, d = _random_inputs(B, K, V, torch.float32, seed=3, match_p=1.0)
    d[0, 1] = V
    d[1, 0] = -7
    ocm = Ocm(256, 0)
    mem = ORACLE.OCM(256, 0)
    buf = StepBuffers(B, K, V, torch.float32, diag=True)
    csd_step(z, d, ocm, 0.0, buf)
    ref = oracle_step(z, d, mem, 0.0)
    compare(buf, ref)
    assert buf.accept_len.tolist() == [1, 0]
    st = compare_memory(ocm, mem)
    assert st["flags"] == 2 and st["n_keys"] == 0
    # a NaN logit raises the NaN flag and the launch still completes
    z[1, 2, 17] = float("nan")
    csd_verify(z, d.clamp(0, V - 1), ocm, 0.0, buf)
    torch.cuda.synchronize()
    assert ocm.stats()["flags"] & 1
    ocm.close()


def test_verify_leaves_memory_alone_and_is_deterministic():
    wl = dataclasses.replace(WORKLOADS["batched_serving"], B=4)
    syn = Synth(wl, 1, "cuda")
    ocm = Ocm(4096, 1)
    z, d = syn.step(0)
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
    csd_step(z, d, ocm, 0.3, buf)
    before = [x.clone() for x in ocm.export()]
    csd_verify(z, d, ocm, 0.3, buf)
    first = {k: v.clone() for k, v in buf.diag.items()}
    outs = [buf.accept_len.clone(), buf.next_token.clone(), buf.rescued_mask.clone()]
    csd_verify(z, d, ocm, 0.3, buf)
    after = ocm.export()
    assert all(torch.equal(a, b) for a, b in zip(before, after))
    for k, v in buf.diag.items():                       # bit-identical, including the sums
        assert torch.equal(v.view(torch.int32), first[k].view(torch.int32)), k
    assert torch.equal(outs[0], buf.accept_len) and torch.equal(outs[1], buf.next_token)
    assert torch.equal(outs[2], buf.rescued_mask)
    ocm.close()


# ---------------------------------------------------------------------------------------
# lock-step runs of the five workloads (bounded step counts; the oracle is the slow side)
# ---------------------------------------------------------------------------------------
def test_workload_tiny_lockstep():
    tot, near, st = lockstep(WORKLOADS["tiny"], steps=1000, tau=0.3, check_every=250)
    assert st["rescues"] == tot["resc"] and tot["resc"] > 0
    print(f"tiny: accepted {tot['acc']} rescued {tot['resc']} near-ties {near} keys {st['n_keys']}")


@pytest.mark.parametrize("tau", [0.1, 0.3, 0.5])
def test_workload_single_stream_lockstep(tau):
    wl = WORKLOADS["single_stream"]
    tot, near, st = lockstep(wl, steps=150, tau=tau, prewarm_pairs=4000)
    assert tot["resc"] > 0
    print(f"single_stream tau={tau}: accepted {tot['acc']} rescued {tot['resc']} near-ties {near}")


def test_workload_batched_serving_lockstep():
    tot, near, st = lockstep(WORKLOADS["batched_serving"], steps=12, tau=0.3, lam=2)
    assert tot["resc"] > 0
    print(f"batched_serving: accepted {tot['acc']} rescued {tot['resc']} near-ties {near}")


@pytest.mark.parametrize("tau", [0.2, 0.4])
def test_workload_large_batch_lockstep(tau):
    wl = WORKLOADS["large_batch"]
    tot, near, st = lockstep(wl, steps=2, tau=tau, prewarm_pairs=200000, diag=True)
    assert tot["resc"] > 0
    print(f"large_batch tau={tau}: accepted {tot['acc']} rescued {tot['resc']} near-ties {near}")


def test_workload_ocm_contention_lockstep():
    wl = WORKLOADS["ocm_contention"]
    tot, near, st = lockstep(wl, steps=16, tau=0.3, check_every=4)
    assert tot["resc"] > 0
    print(f"ocm_contention: accepted {tot['acc']} rescued {tot['resc']} near-ties {near} keys {st['n_keys']}")


@pytest.mark.parametrize("name,steps,tau", [("tiny", 60, 0.3), ("single_stream", 30, 0.1), ("batched_serving", 6, 0.3),
                                             ("large_batch", 2, 0.2), ("ocm_contention", 6, 0.3)])
def test_lockstep_in_the_benchmark_launch_shape(name, steps, tau):
    """The full-size workloads once more in the launch configuration bench.py times: step
    overlap on, hence one block per SM and launch and programmatic launches."""
    from paper_2604_13634_b200 import csd_set_overlap
    wl = WORKLOADS[name]
    try:
        csd_set_overlap(True)
        shape = csd_launch_shape(wl.B, wl.K, wl.V, CSD_F32 if wl.dtype == "f32" else CSD_BF16)
        assert shape["grid"] <= torch.cuda.get_device_properties(0).multi_processor_count
        tot, near, st = lockstep(wl, steps=steps, tau=tau, lam=2, prewarm_pairs=2000)
        assert tot["resc"] > 0
    finally:
        csd_set_overlap(False)


def test_contention_fills_the_table():
    """The contention workload with a small table: the run crosses all three update
    regimes (room, canonical admission, full) and the memory still matches the oracle."""
    wl = dataclasses.replace(WORKLOADS["ocm_contention"], B=16, V=32768, ocm_slots=512)
    tot, near, st = lockstep(wl, steps=80, tau=0.3, check_every=1, diag=False)
    assert st["n_keys"] == 256 and st["n_dropped"] > 0


@pytest.mark.parametrize("overlap", [False, True], ids=["alone", "overlap"])
def test_one_batch_row_fills_the_table(overlap):
    """One batch row (the paper's own setting): the launch's only finalising warp takes no global ticket and adds
    from the slots its own look-ups left.  A table far too small takes the run through all three update regimes;
    the memory, its key count and every step match the oracle."""
    from paper_2604_13634_b200 import csd_set_overlap
    wl = dataclasses.replace(WORKLOADS["ocm_contention"], B=1, K=8, V=32768, ocm_slots=128)
    try:
        csd_set_overlap(overlap)
        tot, near, st = lockstep(wl, steps=400, tau=0.3, check_every=1, diag=False)
    finally:
        csd_set_overlap(False)
    assert st["n_keys"] == 64 and st["n_dropped"] > 0 and tot["resc"] > 0


# ---------------------------------------------------------------------------------------
# the memory on its own
# ---------------------------------------------------------------------------------------
def test_update_kernel_regimes_and_import_export():
    g = torch.Generator(device="cuda").manual_seed(5)
    for n_slots, n, vocab in ((1 << 16, 200000, 300), (256, 5000, 40), (1024, 3000, 25), (64, 31, 1000), (64, 40, 1000)):
        ocm = Ocm(n_slots, 6)
        mem = ORACLE.OCM(n_slots, 6)
        for rep in range(3):
            d = torch.randint(0, vocab, (n,), generator=g, device="cuda", dtype=torch.int32)
            t = torch.randint(0, vocab, (n,), generator=g, device="cuda", dtype=torch.int32)
            d[::17] = -1                                    # placeholders are skipped
            ocm.update(d, t)
            mem.update(zip(d.cpu().tolist(), t.cpu().tolist()))
            compare_memory(ocm, mem)
        # export -> fresh table -> import reproduces the contents
        d, t, c = ocm.export()
        other = Ocm(n_slots, 6)
        other.import_(d.to(torch.int32).cuda(), t.to(torch.int32).cuda(), c.to(torch.int32).cuda())
        d2, t2, c2 = other.export()
        assert torch.equal(d, d2) and torch.equal(t, t2) and torch.equal(c, c2)
        # saturation
        one = torch.tensor([int(d[0])], dtype=torch.int32, device="cuda")
        two = torch.tensor([int(t[0])], dtype=torch.int32, device="cuda")
        big = torch.tensor([-2], dtype=torch.int32, device="cuda")          # 2^32 - 2 as bits
        other.import_(one, two, big)
        other.import_(one, two, big)
        d3, t3, c3 = other.export()
        assert int(c3[0]) == 2**32 - 1 and other.stats()["flags"] & 8
        other.reset()
        assert other.stats()["n_keys"] == 0 and other.export()[0].numel() == 0
        ocm.close(); other.close()


def test_memory_survives_a_file(tmp_path):
    """Calibration hands its table to deployment through a file (Sec. 4.2, Phase 1): csd_ocm_save, csd_ocm_load,
    same triples, same lambda; the bytes on disk are the documented layout; a smaller table admits the saved pairs
    in sorted order up to its own limit; a damaged file is refused."""
    import struct
    from paper_2604_13634_b200 import CsdError
    g = torch.Generator(device="cuda").manual_seed(11)
    ocm = Ocm(4096, 3)
    d = torch.randint(0, 50, (5000,), generator=g, device="cuda", dtype=torch.int32)
    t = torch.randint(0, 50, (5000,), generator=g, device="cuda", dtype=torch.int32)
    ocm.update(d, t)
    mem = ORACLE.OCM(4096, 3)
    mem.update(zip(d.cpu().tolist(), t.cpu().tolist()))
    path = str(tmp_path / "table.ocm")
    ocm.save(path)
    raw = open(path, "rb").read()
    magic, version, lam, n_slots, n, n_dropped = struct.unpack_from("<8sIIQQQ", raw, 0)
    assert (magic, version, lam, n_slots, n, n_dropped) == (b"CSDOCM\0\0", 1, 3, 4096, mem.n_keys, mem.n_dropped)
    assert raw[40:64] == bytes(24) and len(raw) == 64 + 12 * n
    rec = np.frombuffer(raw, dtype=np.dtype([("d", "<i4"), ("t", "<i4"), ("c", "<u4")]), offset=64)
    rd, rt, rc = mem.export()
    assert np.array_equal(rec["d"], rd) and np.array_equal(rec["t"], rt) and np.array_equal(rec["c"], rc)
    back = Ocm.load(path)
    assert all(torch.equal(a, b) for a, b in zip(ocm.export(), back.export()))
    assert back.stats()["lambda"] == 3 and back.n_slots == 4096
    small = Ocm.load(path, n_slots=256)
    sd, st_, sc = small.export()
    fd, ft, fc = ocm.export()
    assert small.stats()["n_keys"] == 128 and small.stats()["n_dropped"] == len(fd) - 128
    assert torch.equal(sd, fd[:128]) and torch.equal(st_, ft[:128]) and torch.equal(sc, fc[:128])
    for damaged in (raw[:40], b"X" + raw[1:], raw[:64] + raw[76:88] + raw[64:76] + raw[88:], raw[:-5]):
        open(path, "wb").write(damaged)
        with pytest.raises(CsdError):
            Ocm.load(path)
    with pytest.raises(CsdError):
        Ocm.load(str(tmp_path / "missing.ocm"))
    for o in (ocm, back, small):
        o.close()


def test_merge_of_overlapping_weighted_tables():
    """Two tables with common and distinct pairs: dst += src equals the oracle's merge (update with the
    source's sorted triples as weighted entries), with room for everything and across the capacity limit."""
    g = torch.Generator(device="cuda").manual_seed(12)
    for dst_slots, vocab in ((4096, 40), (256, 40), (64, 12)):
        a, b = Ocm(dst_slots, 2), Ocm(4096, 2)
        ma, mb = ORACLE.OCM(dst_slots, 2), ORACLE.OCM(4096, 2)
        for ocm, mem, n, lo in ((a, ma, 700, 0), (b, mb, 3000, vocab // 3)):
            d = torch.randint(lo, lo + vocab, (n,), generator=g, device="cuda", dtype=torch.int32)
            t = torch.randint(lo, lo + vocab, (n,), generator=g, device="cuda", dtype=torch.int32)
            ocm.update(d, t)
            mem.update(zip(d.cpu().tolist(), t.cpu().tolist()))
        common = set(ma.table) & set(mb.table)
        assert common and set(mb.table) - set(ma.table)
        a.merge(b)
        ma.merge(mb)
        st = compare_memory(a, ma)
        compare_memory(b, mb)                                   # the source is unchanged
        if dst_slots < 4096:
            assert st["n_keys"] == dst_slots // 2 and st["n_dropped"] > 0
        a.merge(b); ma.merge(mb)                                # once more: now every admitted pair is common
        compare_memory(a, ma)
        a.close(); b.close()


def test_ageing_matches_the_oracle():
    """csd_ocm_age on its own, and inside a run of the contention workload with a 512-slot table that is aged
    every 40 steps: the table fills, ageing frees room, new pairs are admitted again, and the memory equals the oracle's after every step."""
    g = torch.Generator(device="cuda").manual_seed(13)
    for n_slots, n, vocab in ((1 << 14, 20000, 90), (64, 200, 7), (256, 3000, 30)):
        ocm, mem = Ocm(n_slots, 1), ORACLE.OCM(n_slots, 1)
        for rep in range(4):
            d = torch.randint(0, vocab, (n,), generator=g, device="cuda", dtype=torch.int32)
            t = torch.randint(0, vocab, (n,), generator=g, device="cuda", dtype=torch.int32)
            ocm.update(d, t); mem.update(zip(d.cpu().tolist(), t.cpu().tolist()))
            compare_memory(ocm, mem)
            ocm.age(); mem.age()
            compare_memory(ocm, mem)
        for _ in range(34):                                     # down to nothing
            ocm.age(); mem.age()
        assert compare_memory(ocm, mem)["n_keys"] == 0
        ocm.close()
    wl = dataclasses.replace(WORKLOADS["ocm_contention"], B=16, V=32768, ocm_slots=512)
    syn = Synth(wl, 0, "cuda")
    ocm, mem = Ocm(wl.ocm_slots, wl.lam), ORACLE.OCM(wl.ocm_slots, wl.lam)
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
    full_seen = forgotten = 0
    for s in range(160):
        z, d = syn.step(s)
        csd_step(z, d, ocm, 0.3, buf)
        compare(buf, oracle_step(z, d, mem, 0.3))
        full_seen += mem.n_keys == mem.limit
        if (s + 1) % 40 == 0:
            before = mem.n_keys
            ocm.age(); mem.age()
            forgotten += before - mem.n_keys
        compare_memory(ocm, mem)
    st = ocm.stats()
    assert full_seen > 0 and forgotten > 100 and st["rescues"] > 0 and st["flags"] == 0
    ocm.close()


def test_host_entry_point_matches_device_entry_point():
    wl = dataclasses.replace(WORKLOADS["batched_serving"], B=6)
    syn = Synth(wl, 2, "cuda")
    a, b = Ocm(4096, 1), Ocm(4096, 1)
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype)
    host = HostStep(wl.B, wl.K, wl.V, wl.torch_dtype)
    for s in range(5):
        z, d = syn.step(s)
        csd_step(z, d, a, 0.3, buf)
        acc, nxt, resc = host(z.cpu().pin_memory(), d.cpu().pin_memory(), b, 0.3)
        assert torch.equal(acc, buf.accept_len.cpu()) and torch.equal(nxt, buf.next_token.cpu())
        assert torch.equal(resc, buf.rescued_mask.cpu())
    assert all(torch.equal(x, y) for x, y in zip(a.export(), b.export()))
    a.close(); b.close()


@pytest.mark.parametrize("chunk_bytes,ctas,threads", [(512, 4, 256), (4096, 1, 1024), (8192, 2, 512), (36864, 3, 96),
                                                        (1 << 20, 4, 32), (16384, 8, 128)])
def test_parity_under_other_splits(chunk_bytes, ctas, threads):
    try:
        csd_set_tuning(chunk_bytes, ctas, threads)
        wl = dataclasses.replace(WORKLOADS["ocm_contention"], B=8)
        shape = csd_launch_shape(wl.B, wl.K, wl.V, CSD_BF16)
        assert shape["block"] == threads and shape["grid"] <= 148 * ctas and shape["chunk_elems"] * 2 >= chunk_bytes
        lockstep(wl, steps=3, tau=0.3, lam=1)
        wl = dataclasses.replace(WORKLOADS["large_batch"], B=4)
        lockstep(wl, steps=2, tau=0.2, lam=1)
    finally:
        csd_set_tuning(0, 0, 0)


def test_many_short_rows_per_warp():
    """Many short rows: a block's span covers far more than 32 rows and several batch rows, so
    it works through several windows, publishing after each."""
    for (B, K, V, dtype) in ((600, 3, 160, torch.float32), (97, 32, 520, torch.bfloat16), (30000, 1, 24, torch.bfloat16)):
        for tuning in ((0, 0, 0), (512, 1, 64)):
            try:
                csd_set_tuning(*tuning)
                z, d = _random_inputs(B, K, V, dtype, seed=21)
                ocm = Ocm(1 << 14, 0)
                mem = ORACLE.OCM(1 << 14, 0)
                buf = StepBuffers(B, K, V, dtype, diag=True)
                csd_step(z, d, ocm, 0.02, buf)
                compare(buf, oracle_step(z, d, mem, 0.02))
                compare_memory(ocm, mem)
                ocm.close()
            finally:
                csd_set_tuning(0, 0, 0)


def test_overlapped_launches_match():
    """Hundreds of back-to-back steps launched with programmatic stream serialization (the
    setting the benchmark times), eagerly and as a replayed CUDA graph, give the same
    results as plain launches, and the plain run equals the oracle at EVERY step (accepted
    lengths, next tokens, masks, rejection lists, arg-max, counts).  With one set of output
    buffers per step consecutive launches differ in their outputs, so each waits for its
    predecessor to retire, and every step's outputs survive to be compared; with a single
    set they chain on the completion count in the workspace (the path the benchmark takes)
    and the last step, the memory and the statistics are compared."""
    from paper_2604_13634_b200 import csd_set_overlap
    wl = WORKLOADS["batched_serving"]
    syn = Synth(wl, 4, "cuda")
    inputs = [syn.step(s) for s in range(5)]         # an odd ring: replays follow each other out of phase
    reps = 41
    n_steps = reps * len(inputs)

    def run(overlap, graph, one_buffer):
        try:
            csd_set_overlap(overlap)
            ocm = Ocm(wl.ocm_slots, 2)
            ws = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype)         # one shared workspace, as the benchmark has
            if one_buffer:
                bufs = [StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)] * n_steps
            else:
                bufs = [StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True) for _ in range(n_steps)]
            for b in bufs:
                b.workspace, b.ws_bytes = ws.workspace, ws.ws_bytes

            def steps(lo, hi):
                for s in range(lo, hi):
                    z, d = inputs[s % len(inputs)]
                    csd_step(z, d, ocm, 0.3, bufs[s])
            if graph and one_buffer:                 # one ring pass captured, replayed (reps - 1) times
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    steps(0, len(inputs))
                torch.cuda.current_stream().wait_stream(side)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    steps(0, len(inputs))
                for _ in range(reps - 1):
                    g.replay()
            elif graph:                               # the first pass eagerly, all the rest as ONE graph
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    steps(0, len(inputs))
                torch.cuda.current_stream().wait_stream(side)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    steps(len(inputs), n_steps)
                g.replay()
            else:
                steps(0, n_steps)
            torch.cuda.synchronize()
            keep = bufs[-len(inputs):] if one_buffer else bufs
            out = ([(b.accept_len.clone(), b.next_token.clone(), b.rescued_mask.clone(), b.rej_draft.clone(),
                     b.rej_target.clone(), b.diag["t"].clone(), b.diag["cnt"].clone(), b.diag["s"].clone())
                    for b in keep], ocm.export(), ocm.stats())
            ocm.close()
            return out
        finally:
            csd_set_overlap(False)

    plain = {}
    for one_buffer in (False, True):
        ref_out, ref_exp, ref_st = run(False, False, one_buffer)
        plain[one_buffer] = (ref_out, ref_exp)
        assert ref_st["steps"] == n_steps and ref_st["flags"] == 0
        for overlap, graph in ((True, False), (True, True), (False, True)):
            out, exp, st = run(overlap, graph, one_buffer)
            assert st == ref_st, (overlap, graph, one_buffer, st, ref_st)
            assert all(torch.equal(p, q) for p, q in zip(exp, ref_exp)), (overlap, graph, one_buffer)
            assert len(out) == len(ref_out)
            for x, y in zip(out, ref_out):
                assert all(torch.equal(p, q) for p, q in zip(x[:-1], y[:-1])), (overlap, graph, one_buffer)
                # the launch shape, and with it the summation tree, depends on the overlap setting
                assert torch.allclose(x[-1], y[-1], rtol=1e-5, atol=0), (overlap, graph, one_buffer)
    # the plain run against the oracle: every step of the per-step run, the last step of the single-buffer run
    mem = ORACLE.OCM(wl.ocm_slots, 2)
    per_step, _ = plain[False]
    last_pass, _ = plain[True]
    for s in range(n_steps):
        z, d = inputs[s % len(inputs)]
        ref = oracle_step(z, d, mem, 0.3)
        got = per_step[s]
        for k, name in enumerate(("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target", "t")):
            assert np.array_equal(got[k].cpu().numpy(), ref[name]), (s, name)
        assert np.array_equal(got[6].cpu().numpy().astype(np.int64) & 0xFFFFFFFF, ref["cnt"]), (s, "cnt")
        if s == n_steps - 1:                      # a single set of buffers keeps the last step only
            got = last_pass[-1]
            for k, name in enumerate(("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target", "t")):
                assert np.array_equal(got[k].cpu().numpy(), ref[name]), (s, name, "single buffer")
    rd, rt, rc = mem.export()
    for _, exp in plain.values():
        assert np.array_equal(exp[0].numpy(), rd) and np.array_equal(exp[1].numpy(), rt) and np.array_equal(exp[2].numpy(), rc)


def test_launch_shape_changes_on_a_live_workspace():
    """csd_set_overlap and csd_set_tuning change the layout of the scratch inside a workspace.  A
    workspace that has seen steps of one layout is cleared by the library before a step of another
    layout uses it, so switching on a live workspace gives the same results as a fresh one."""
    from paper_2604_13634_b200 import csd_set_overlap
    wl = WORKLOADS["batched_serving"]
    syn = Synth(wl, 6, "cuda")
    ocm = Ocm(wl.ocm_slots, 1)
    mem = ORACLE.OCM(wl.ocm_slots, 1)
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
    settings = [(False, (0, 0, 0)), (True, (0, 0, 0)), (False, (0, 0, 0)), (False, (8192, 2, 128)), (True, (0, 0, 0)),
                (True, (4096, 3, 256)), (False, (0, 0, 0))]
    try:
        for s, (overlap, tuning) in enumerate(settings):
            csd_set_overlap(overlap)
            csd_set_tuning(*tuning)
            for rep in range(3):
                z, d = syn.step(2 * s + rep % 2)
                csd_step(z, d, ocm, 0.3, buf)
                compare(buf, oracle_step(z, d, mem, 0.3))
        st = compare_memory(ocm, mem)
        assert st["flags"] == 0 and st["steps"] == 3 * len(settings)
    finally:
        csd_set_overlap(False)
        csd_set_tuning(0, 0, 0)
    ocm.close()


def test_bounds_checked_build_runs_the_small_shapes_clean():
    """The same sources built with -DCSD_DEBUG compare every index they compute with its bound (a failed
    check skips the access and raises CSD_FLAG_INTERNAL; nothing traps).  The small-shape parity tests
    run once more against that build, in a process of their own, and the flag must stay clear."""
    import os
    import subprocess
    import sys
    from paper_2604_13634_b200 import build
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    assert os.path.exists(build.LIB_DEBUG), "libcsd_debug.so has not been built"
    env = dict(os.environ, CSD_DEBUG="1")
    sel = ("test_elementwise_parity_small or test_many_short_rows_per_warp or test_contention_fills_the_table "
           "or test_strided_and_misaligned_views or test_internal_flag_is_clear")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", sel,
                        os.path.join(root, "tests", "test_gpu_parity.py"), os.path.join(root, "tests", "test_gpu_sampled_parity.py")],
                       cwd=root, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:]


def test_internal_flag_is_clear():
    """A step on each dtype and path; the library's own index checks (all of them in the CSD_DEBUG build,
    the partial-slot check in every build) must not have fired."""
    from paper_2604_13634_b200 import binding
    for (B, K, V, dtype) in ((7, 5, 33000, torch.float32), (9, 3, 40001, torch.bfloat16), (300, 2, 700, torch.bfloat16)):
        z, d = _random_inputs(B, K, V, dtype, seed=5)
        ocm = Ocm(1 << 12, 1)
        buf = StepBuffers(B, K, V, dtype)
        for _ in range(3):
            csd_step(z, d, ocm, 0.01, buf)
        st = ocm.stats()
        assert st["flags"] & binding.FLAG_INTERNAL == 0 and st["debug_site"] == 0, st
        ocm.close()
    want = "libcsd_debug.so" if os.environ.get("CSD_DEBUG", "0") not in ("", "0") else "libcsd.so"
    assert binding.LIB_PATH.endswith(want)


def test_long_rows():
    """Rows of 4 MiB: each is shared by several blocks, and a block's span needs larger chunks.
    The second case has so many units and blocks that the span arithmetic leaves 32 bits."""
    for (B, tuning) in ((48, (0, 0, 0)), (64, (0, 32, 128))):
        try:
            csd_set_tuning(*tuning)
            K, V = 1, 1 << 20
            z, d = _random_inputs(B, K, V, torch.float32, seed=11)
            ocm = Ocm(256, 0)
            mem = ORACLE.OCM(256, 0)
            buf = StepBuffers(B, K, V, torch.float32, diag=True)
            csd_step(z, d, ocm, 0.01, buf)
            compare(buf, oracle_step(z, d, mem, 0.01))
            compare_memory(ocm, mem)
            ocm.close()
            del z, d, buf
            torch.cuda.empty_cache()
        finally:
            csd_set_tuning(0, 0, 0)
