"""The entry point that allocates nothing (collected last on purpose).

csd_verify_static is for callers that cannot obtain device memory when they need to verify
a step -- a server whose framework took the whole GPU for its pool at start-up, a plug-in
without an allocator, a loop where an allocation may stall or fail.  It keeps the kernel's
scratch in a fixed array inside the library.  This test calls it through the C ABI, twice in
a row and with a different shape the second time (the array is shared and keeps the previous
call's contents), and checks every output against the ordinary csd_verify on the same inputs:
same kernel, same shape, so the results must be identical bit for bit.
"""

import ctypes

import pytest
import torch

from paper_2604_13634_b200 import Ocm, StepBuffers, binding, csd_step, csd_verify
from synth_inputs import WORKLOADS, Synth
import dataclasses

pytestmark = pytest.mark.gpu


def _call_static(L, z, d, ocm, tau, buf):
    B, K1, V = z.shape
    rc = L.csd_verify_static(z.data_ptr(), buf.dtype_code, B, K1 - 1, V, z.stride(0), z.stride(1), d.data_ptr(),
                             ocm.handle, ctypes.c_float(tau), buf.accept_len.data_ptr(), buf.next_token.data_ptr(),
                             buf.rescued_mask.data_ptr(), buf.rej_draft.data_ptr(), buf.rej_target.data_ptr(),
                             ctypes.byref(buf._diag_struct), torch.cuda.current_stream().cuda_stream)
    assert rc == 0, L.csd_status_string(rc)


def _snapshot(buf):
    torch.cuda.synchronize()
    out = [buf.accept_len.clone(), buf.next_token.clone(), buf.rescued_mask.clone(), buf.rej_draft.clone(),
           buf.rej_target.clone()]
    out += [v.clone().view(torch.int32) for v in buf.diag.values()]
    return out


def test_static_scratch_entry_point_matches_csd_verify():
    L = binding.lib()
    shapes = [dataclasses.replace(WORKLOADS["batched_serving"], B=8),        # bf16, several blocks per row
              dataclasses.replace(WORKLOADS["large_batch"], B=6, K=4)]        # fp32, another layout of the scratch
    for rep in range(2):                                                      # two rounds: the array is reused
        for wl in shapes:
            syn = Synth(wl, seed=10 + rep, device="cuda")
            ocm = Ocm(4096, lam=1)
            warm = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype)
            z, d = syn.step(0)
            csd_step(z, d, ocm, 0.3, warm)                                     # put some pairs into the memory
            for s in (0, 1):                                                   # two calls in a row per shape
                z, d = syn.step(s)
                ref_buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
                csd_verify(z, d, ocm, 0.3, ref_buf)
                ref = _snapshot(ref_buf)
                got_buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
                _call_static(L, z, d, ocm, 0.3, got_buf)
                got = _snapshot(got_buf)
                for a, b in zip(got, ref):
                    assert torch.equal(a, b)
                assert int(ref_buf.rescued_mask.sum()) + int((ref_buf.accept_len > 0).sum()) > 0
            ocm.close()


def test_static_scratch_entry_point_takes_no_device_memory():
    """What the entry point is for: the free device memory reported by the driver is the same before
    and after a series of calls (inputs, outputs and the memory object were allocated beforehand)."""
    L = binding.lib()
    wl = dataclasses.replace(WORKLOADS["batched_serving"], B=8)
    syn = Synth(wl, seed=3, device="cuda")
    ocm = Ocm(4096, lam=1)
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
    z, d = syn.step(0)
    _call_static(L, z, d, ocm, 0.3, buf)          # the first call on a device looks up the array's address
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(5):
        _call_static(L, z, d, ocm, 0.3, buf)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    ocm.close()


def test_static_scratch_refuses_what_does_not_fit():
    L = binding.lib()
    one = ctypes.c_void_p(256)
    ocm = Ocm(256, lam=1)
    # 40 000 batch rows of 2 logit rows: the scratch this needs is far beyond the fixed array
    assert binding.csd_workspace_bytes(40000, 1, 4096, 0) > binding.STATIC_SCRATCH_BYTES
    rc = L.csd_verify_static(one, 0, 40000, 1, 4096, 2 * 4096, 4096, one, ocm.handle, ctypes.c_float(0.3),
                             one, one, one, one, one, None, None)
    assert rc == 5
    rc = L.csd_verify_static(one, 0, 2, 40, 4096, 41 * 4096, 4096, one, ocm.handle, ctypes.c_float(0.3),
                             one, one, one, one, one, None, None)
    assert rc == 4
    ocm.close()
