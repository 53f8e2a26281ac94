"""CPU-side checks of the C ABI: the library loads, exports what the header declares,
and its host logic (argument checks, threshold, launch shapes) behaves as documented."""

import ctypes
import os
import re

import numpy as np
import pytest

from oracle import csd_oracle as ORACLE
from paper_2604_13634_b200 import binding, build


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def _declared(repo_root):
    text = open(os.path.join(repo_root, "include", "csd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(csd_[a-z_0-9]+)\s*\(", text)))


def test_exports_match_header(L, repo_root):
    names = _declared(repo_root)
    assert len(names) >= 18
    for n in names:
        assert hasattr(L, n), f"{n} declared in csd.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_threshold_matches_oracle(L):
    taus = [0.0, 1e-10, 0.001, 0.01, 0.05, 0.1, 0.2, 0.25, 0.3, 0.4, 0.5, 0.6, 0.9, 1.0, 1.5, 7.0]
    taus += list(np.random.default_rng(0).random(2000).astype(np.float32))
    for tau in taus:
        assert binding.csd_scg_threshold(float(tau)) == ORACLE.scg_threshold(float(tau)), tau


def test_status_strings(L):
    seen = {L.csd_status_string(i) for i in range(6)}
    assert len(seen) == 6 and b"ok" in seen


SHAPES = ((1, 4, 32000, 0), (1, 8, 128256, 1), (32, 5, 151936, 1), (128, 8, 128256, 0), (64, 6, 152064, 1),
          (3, 1, 7, 0), (2, 32, 1000, 1), (1, 1, 1 << 22, 0), (5, 2, 70001, 0), (48, 1, 1 << 20, 0), (30000, 1, 24, 1))


def test_shapes_and_workspace(L):
    for (B, K, V, dt) in SHAPES:
        s = binding.csd_launch_shape(B, K, V, dt)
        eb = 4 if dt == 0 else 2
        rows = B * (K + 1)
        units = rows * -(-V * eb // 512)
        assert s["block"] == 256 and 1 <= s["grid"] <= min(148 * 4, units, 64 * rows)
        assert (s["chunk_elems"] * eb) % 512 == 0 and 1 <= s["parts_per_row"] <= 66
        ws = binding.csd_workspace_bytes(B, K, V, dt)
        assert ws >= 2 * (rows * s["parts_per_row"] * 16 + 4 * B * K + 4 * B + 4) + 12
        assert binding.csd_host_staging_bytes(B, K, V, dt) >= rows * V * eb + ws
    assert binding.csd_workspace_bytes(0, 4, 100, 0) == 0
    assert binding.csd_workspace_bytes(1, 33, 100, 0) == 0
    assert binding.csd_workspace_bytes(1, 4, 100, 7) == 0


def test_even_split_geometry():
    """Host replay of the kernels' span arithmetic: every span is non-empty, the blocks touching
    a row are consecutive and fit the row's slots, and a span never needs more chunk results
    than a block can hold."""
    for (B, K, V, dt) in SHAPES:
        s = binding.csd_launch_shape(B, K, V, dt)
        eb = 4 if dt == 0 else 2
        U = -(-V * eb // 512)
        rows = B * (K + 1)
        T, G = rows * U, s["grid"]
        CH = s["chunk_elems"] * eb // 512
        begin = [c * T // G for c in range(G + 1)]
        assert all(begin[c + 1] > begin[c] for c in range(G))
        assert max(begin[c + 1] - begin[c] for c in range(G)) // CH + 34 <= 1024
        owner = lambda g: ((g + 1) * G - 1) // T
        for r in list(range(min(rows, 40))) + [rows - 1]:
            first, last = owner(r * U), owner((r + 1) * U - 1)
            assert begin[first] <= r * U < begin[first + 1] and begin[last] <= (r + 1) * U - 1 < begin[last + 1]
            assert last - first + 1 <= s["parts_per_row"]


def test_argument_checks_refuse_before_launch(L):
    null = None
    one = ctypes.c_void_p(16)      # a non-null, never dereferenced, address
    f = ctypes.c_float
    def verify(**kw):
        a = dict(logits=one, dt=0, B=2, K=3, V=64, sb=4 * 64, sk=64, draft=one, ocm=one, tau=0.3, acc=one, nxt=one,
                 resc=one, rd=one, rt=one, diag=None, ws=one, wsb=1 << 20)
        a.update(kw)
        return L.csd_verify(a["logits"], a["dt"], a["B"], a["K"], a["V"], a["sb"], a["sk"], a["draft"], a["ocm"],
                            f(a["tau"]), a["acc"], a["nxt"], a["resc"], a["rd"], a["rt"], a["diag"], a["ws"],
                            a["wsb"], None)
    assert verify(logits=null) == 1 and verify(draft=null) == 1 and verify(ocm=null) == 1 and verify(ws=null) == 1
    assert verify(B=0) == 1 and verify(K=0) == 1 and verify(V=-5) == 1 and verify(dt=3) == 1
    assert verify(K=33, sb=34 * 64) == 4
    assert verify(tau=float("nan")) == 1 and verify(tau=-0.1) == 1 and verify(tau=float("inf")) == 1
    assert verify(sk=63) == 1 and verify(sb=64) == 1
    assert verify(wsb=16) == 5
    assert verify(ws=ctypes.c_void_p(24)) == 5
    assert L.csd_ocm_update(null, one, one, 4, None) == 1
    assert L.csd_ocm_update(one, null, one, 4, None) == 1
    assert L.csd_ocm_update(one, one, one, -1, None) == 1
    out = ctypes.c_void_p()
    assert L.csd_ocm_create(ctypes.byref(out), 1000, 6, 0) == 1      # not a power of two
    assert L.csd_ocm_create(ctypes.byref(out), 32, 6, 0) == 1
    assert L.csd_ocm_create(None, 1024, 6, 0) == 1
    assert L.csd_ocm_create(ctypes.byref(out), 1 << 31, 6, 0) == 1
    assert L.csd_set_tuning(1000, 0, 0) == 1 and L.csd_set_tuning(0, 33, 0) == 1 and L.csd_set_tuning(0, 0, 48) == 1
    assert L.csd_set_tuning(0, 0, 0) == 0


def test_binding_refuses_without_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("device present")
    with pytest.raises(binding.CsdError):
        binding.Ocm(1024)


def test_plans_of_the_other_entry_points(L):
    """Host-side sizing of the stochastic, two-phase and LM-head steps (no device needed)."""
    for (B, K, V, dt) in SHAPES[:7]:
        assert L.csd_sampled_workspace_bytes(B, K, V, dt) > 0
        if K >= 2:
            ws = L.csd_early_exit_workspace_bytes(B, K, V, dt, 0)
            assert ws >= binding.csd_workspace_bytes(B, max(1, (K + 1) // 3), V, dt) // 2 + 4 * B
            assert L.csd_early_exit_workspace_bytes(B, K, V, dt, K - 1) > 0
        else:
            assert L.csd_early_exit_workspace_bytes(B, K, V, dt, 0) == 0
    # launches of the stochastic step: one round of draws for steps of a few megabytes, two rounds beyond
    L.csd_sampled_launches.argtypes, L.csd_sampled_launches.restype = [ctypes.c_int] * 4, ctypes.c_int
    L.csd_sampled_set_rounds.argtypes, L.csd_sampled_set_rounds.restype = [ctypes.c_int], ctypes.c_int
    assert L.csd_sampled_launches(1, 8, 128256, 1) == 5 and L.csd_sampled_launches(32, 5, 151936, 1) == 7
    assert L.csd_sampled_launches(1, 4, 32000, 0) == 5 and L.csd_sampled_launches(128, 8, 128256, 0) == 7
    assert L.csd_sampled_launches(1, 40, 1000, 0) == 0                       # K beyond the limit
    try:
        assert L.csd_sampled_set_rounds(1) == 0 and L.csd_sampled_launches(128, 8, 128256, 0) == 5
        assert L.csd_sampled_set_rounds(2) == 0 and L.csd_sampled_launches(1, 8, 128256, 1) == 7
        assert L.csd_sampled_set_rounds(3) != 0 and L.csd_sampled_set_rounds(-1) != 0
    finally:
        L.csd_sampled_set_rounds(0)
    g, n, t, per = (ctypes.c_int() for _ in range(4))
    L.csd_lmhead_set_pairing.argtypes, L.csd_lmhead_set_pairing.restype = [ctypes.c_int], ctypes.c_int
    assert L.csd_lmhead_set_pairing(3) != 0 and L.csd_lmhead_set_pairing(-1) != 0
    try:
        for mode in (1, 2):                              # one block per SM; pairs of blocks, a pair's tile twice as wide
            assert L.csd_lmhead_set_pairing(mode) == 0
            for (B, K, H, V) in ((32, 5, 4096, 151936), (64, 6, 4096, 152064), (128, 8, 4096, 128256), (1, 1, 64, 17), (2, 3, 128, 1000)):
                assert L.csd_lmhead_shape(B, K, H, V, ctypes.byref(g), ctypes.byref(n), ctypes.byref(t), ctypes.byref(per)) == 0
                owners = g.value // mode                 # blocks or pairs: each owns `per` consecutive tiles
                assert 1 <= g.value <= 148 and g.value % mode == 0
                assert n.value % (16 * mode) == 0 and 16 * mode <= n.value <= 256 * mode
                assert t.value == -(-V // n.value) and owners * per.value >= t.value and (owners - 1) * per.value < t.value
                assert L.csd_lmhead_workspace_bytes(B, K, H, V) >= B * (K + 1) * g.value * 16 + 4 * B * K
    finally:
        L.csd_lmhead_set_pairing(0)
    assert L.csd_lmhead_workspace_bytes(2, 3, 100, 1000) == 0            # H must be a multiple of 64
    assert L.csd_lmhead_shape(2, 33, 128, 1000, None, None, None, None) != 0
