"""ctypes binding of libcsd.so: argument marshalling only.

Every function mirrors one entry point of include/csd.h under the same name.
Tensors are torch CUDA tensors (device memory and streams are torch's); all
arithmetic happens in the library's kernels.  There is no fallback: if the
library cannot be loaded, or a call fails, an exception is raised.
"""

from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int, c_int64, c_size_t, c_uint32, c_uint64, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# CSD_DEBUG=1 in the environment selects the bounds-checked build of the same sources
LIB_PATH = os.path.join(_HERE, "libcsd_debug.so" if os.environ.get("CSD_DEBUG", "0") not in ("", "0") else "libcsd.so")

CSD_F32, CSD_BF16 = 0, 1
CSD_MAX_K = 32
FLAG_NAN_LOGIT, FLAG_BAD_DRAFT, FLAG_PROBE_EXHAUSTED, FLAG_COUNT_SATURATED, FLAG_INTERNAL = 1, 2, 4, 8, 16

EXPORTS = [
    "csd_ocm_create", "csd_ocm_reset", "csd_ocm_destroy", "csd_ocm_set_lambda",
    "csd_workspace_bytes", "csd_workspace_init", "csd_verify", "csd_ocm_update", "csd_step",
    "csd_host_staging_bytes", "csd_step_host", "csd_verify_static", "csd_ocm_export", "csd_ocm_import", "csd_ocm_stats",
    "csd_scg_threshold", "csd_launch_shape", "csd_set_tuning", "csd_set_overlap", "csd_status_string",
    "csd_sampled_workspace_bytes", "csd_verify_sampled", "csd_step_sampled",
    "csd_ocm_age", "csd_ocm_merge", "csd_ocm_save", "csd_ocm_load", "csd_ocm_set_shared",
    "csd_lmhead_workspace_bytes", "csd_verify_lmhead", "csd_step_lmhead", "csd_lmhead_shape",
    "csd_early_exit_workspace_bytes", "csd_step_early_exit", "csd_lmhead_set_tuning", "csd_lmhead_set_pairing", "csd_lmhead_uses_pairs",
    "csd_sampled_set_rounds", "csd_sampled_launches",
]


class CsdError(RuntimeError):
    pass


class Diag(Structure):
    _fields_ = [(n, c_void_p) for n in ("m", "s", "lse", "t", "zd", "score", "p_d", "p_t", "cnt")]


class SampledDiag(Structure):
    _fields_ = [(n, c_void_p) for n in ("alpha", "accepted", "t_star", "lse_p", "lse_q", "score", "cnt", "bonus")]


class Stats(Structure):
    _fields_ = [(n, c_uint64) for n in ("n_slots", "key_limit", "n_keys", "n_dropped", "steps", "positions",
                                         "matches", "rescues", "rejections")] + [("lambda_", c_uint32), ("flags", c_uint32),
                                                                                 ("debug_site", c_uint32), ("reserved", c_uint32)]

    def as_dict(self):
        d = {n: int(getattr(self, n)) for n, _ in self._fields_}
        d["lambda"] = d.pop("lambda_")
        return d


_lib = None


def lib():
    """The loaded library.  Raises if it has not been built (see build.py)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise CsdError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_13634_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    step_args = [c_void_p, c_int, c_int, c_int, c_int, c_int64, c_int64, c_void_p, c_void_p, c_float,
                 c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, POINTER(Diag), c_void_p, c_size_t, c_void_p]
    sampled_args = [c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_int64, c_int64, c_int64, c_int64, c_void_p, c_void_p,
                    c_uint64, c_float, c_void_p, c_float, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                    POINTER(SampledDiag), c_void_p, c_size_t, c_void_p]
    lmhead_args = [c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_float, c_void_p, c_void_p, c_void_p,
                   c_void_p, c_void_p, POINTER(Diag), c_void_p, c_size_t, c_void_p]
    sigs = {
        "csd_sampled_workspace_bytes": (c_size_t, [c_int, c_int, c_int, c_int]),
        "csd_verify_sampled": (c_int, sampled_args),
        "csd_step_sampled": (c_int, sampled_args),
        "csd_ocm_create": (c_int, [POINTER(c_void_p), c_uint64, c_uint32, c_int]),
        "csd_ocm_reset": (c_int, [c_void_p, c_void_p]),
        "csd_ocm_destroy": (c_int, [c_void_p]),
        "csd_ocm_set_lambda": (c_int, [c_void_p, c_uint32]),
        "csd_workspace_bytes": (c_size_t, [c_int, c_int, c_int, c_int]),
        "csd_workspace_init": (c_int, [c_void_p, c_size_t, c_void_p]),
        "csd_verify": (c_int, step_args),
        "csd_step": (c_int, step_args),
        "csd_verify_static": (c_int, step_args[:-3] + [c_void_p]),
        "csd_ocm_update": (c_int, [c_void_p, c_void_p, c_void_p, c_int64, c_void_p]),
        "csd_host_staging_bytes": (c_size_t, [c_int, c_int, c_int, c_int]),
        "csd_step_host": (c_int, [c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_float,
                                  c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
        "csd_ocm_export": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_uint64, POINTER(c_uint64), c_void_p]),
        "csd_ocm_import": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_uint64, c_void_p]),
        "csd_ocm_stats": (c_int, [c_void_p, POINTER(Stats), c_void_p]),
        "csd_lmhead_workspace_bytes": (c_size_t, [c_int, c_int, c_int, c_int]),
        "csd_verify_lmhead": (c_int, lmhead_args),
        "csd_step_lmhead": (c_int, lmhead_args),
        "csd_lmhead_shape": (c_int, [c_int, c_int, c_int, c_int, POINTER(c_int), POINTER(c_int), POINTER(c_int), POINTER(c_int)]),
        "csd_early_exit_workspace_bytes": (c_size_t, [c_int, c_int, c_int, c_int, c_int]),
        "csd_step_early_exit": (c_int, step_args[:10] + [c_int] + step_args[10:]),
        "csd_lmhead_set_tuning": (c_int, [c_int, c_int]),
        "csd_lmhead_set_pairing": (c_int, [c_int]),
        "csd_sampled_set_rounds": (c_int, [c_int]),
        "csd_sampled_launches": (c_int, [c_int, c_int, c_int, c_int]),
        "csd_lmhead_uses_pairs": (c_int, [c_int, c_int]),
        "csd_ocm_age": (c_int, [c_void_p, c_void_p]),
        "csd_ocm_set_shared": (c_int, [c_void_p, c_int]),
        "csd_ocm_merge": (c_int, [c_void_p, c_void_p, c_void_p]),
        "csd_ocm_save": (c_int, [c_void_p, c_char_p, c_void_p]),
        "csd_ocm_load": (c_int, [POINTER(c_void_p), c_char_p, c_uint64, c_int]),
        "csd_scg_threshold": (c_float, [c_float]),
        "csd_launch_shape": (c_int, [c_int, c_int, c_int, c_int, POINTER(c_int), POINTER(c_int), POINTER(c_int), POINTER(c_int)]),
        "csd_set_tuning": (c_int, [c_int, c_int, c_int]),
        "csd_set_overlap": (c_int, [c_int]),
        "csd_status_string": (c_char_p, [c_int]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


def _check(rc: int, what: str):
    if rc != 0:
        raise CsdError(f"{what}: {lib().csd_status_string(rc).decode()} (status {rc})")


def _stream_ptr(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return CSD_F32
    if t.dtype == torch.bfloat16:
        return CSD_BF16
    raise CsdError(f"logits must be float32 or bfloat16, got {t.dtype}")


def _ptr(t):
    return None if t is None else t.data_ptr()


def csd_scg_threshold(tau: float) -> float:
    return float(lib().csd_scg_threshold(c_float(tau)))


def csd_set_tuning(chunk_bytes: int = 0, ctas_per_sm: int = 0, block_threads: int = 0):
    _check(lib().csd_set_tuning(chunk_bytes, ctas_per_sm, block_threads), "csd_set_tuning")


def csd_set_overlap(enable: bool):
    _check(lib().csd_set_overlap(1 if enable else 0), "csd_set_overlap")


def csd_launch_shape(B, K, V, dtype_code):
    g, b, te, tr = c_int(), c_int(), c_int(), c_int()
    _check(lib().csd_launch_shape(B, K, V, dtype_code, byref(g), byref(b), byref(te), byref(tr)), "csd_launch_shape")
    return dict(grid=g.value, block=b.value, chunk_elems=te.value, parts_per_row=tr.value)


def csd_workspace_bytes(B, K, V, dtype_code) -> int:
    return int(lib().csd_workspace_bytes(B, K, V, dtype_code))


def csd_host_staging_bytes(B, K, V, dtype_code) -> int:
    return int(lib().csd_host_staging_bytes(B, K, V, dtype_code))


class Ocm:
    """Owner of one csd_ocm_t (the Online Correction Memory of Sec. 4.2)."""

    def __init__(self, n_slots: int, lam: int = 6, device: int = 0):
        if not torch.cuda.is_available():
            raise CsdError("a CUDA device is required")
        h = c_void_p()
        _check(lib().csd_ocm_create(byref(h), n_slots, lam, device), "csd_ocm_create")
        self.handle = h
        self.n_slots = n_slots
        self.device = torch.device("cuda", device)

    def close(self):
        if getattr(self, "handle", None):
            torch.cuda.synchronize()
            lib().csd_ocm_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self, stream=None):
        _check(lib().csd_ocm_reset(self.handle, _stream_ptr(stream)), "csd_ocm_reset")

    def set_lambda(self, lam: int):
        _check(lib().csd_ocm_set_lambda(self.handle, lam), "csd_ocm_set_lambda")

    def update(self, rej_draft: torch.Tensor, rej_target: torch.Tensor, stream=None):
        assert rej_draft.dtype == torch.int32 and rej_target.dtype == torch.int32
        assert rej_draft.is_cuda and rej_target.is_cuda and rej_draft.is_contiguous() and rej_target.is_contiguous()
        assert rej_draft.numel() == rej_target.numel()
        _check(lib().csd_ocm_update(self.handle, _ptr(rej_draft), _ptr(rej_target), rej_draft.numel(),
                                    _stream_ptr(stream)), "csd_ocm_update")

    def import_(self, d: torch.Tensor, t: torch.Tensor, cnt: torch.Tensor, stream=None):
        """cnt holds unsigned 32-bit counts; an int32 tensor carrying the same bits is accepted."""
        assert d.dtype == torch.int32 and t.dtype == torch.int32 and cnt.dtype in (torch.int32, torch.uint32)
        assert d.is_cuda and t.is_cuda and cnt.is_cuda
        _check(lib().csd_ocm_import(self.handle, _ptr(d.contiguous()), _ptr(t.contiguous()), _ptr(cnt.contiguous()),
                                    d.numel(), _stream_ptr(stream)), "csd_ocm_import")

    def export(self, stream=None):
        """(d, t, cnt) int64 CPU tensors of the stored pairs, sorted by (d, t).  Synchronises."""
        st = self.stats(stream)
        cap = max(1, st["n_keys"])
        d = torch.empty(cap, dtype=torch.int32, device=self.device)
        t = torch.empty(cap, dtype=torch.int32, device=self.device)
        c = torch.empty(cap, dtype=torch.int32, device=self.device)
        n = c_uint64()
        _check(lib().csd_ocm_export(self.handle, _ptr(d), _ptr(t), _ptr(c), cap, byref(n), _stream_ptr(stream)),
               "csd_ocm_export")
        k = min(int(n.value), cap)
        d = d[:k].cpu().to(torch.int64)
        t = t[:k].cpu().to(torch.int64)
        c = c[:k].cpu().to(torch.int64) & 0xFFFFFFFF
        order = torch.argsort(d * (1 << 32) + t)
        return d[order], t[order], c[order]

    def set_shared(self, enable: bool):
        """Allow steps and updates on different streams to run on this memory at the same time."""
        _check(lib().csd_ocm_set_shared(self.handle, 1 if enable else 0), "csd_ocm_set_shared")

    def age(self, stream=None):
        """Halve every count (rounding down) and forget the pairs that reach zero."""
        _check(lib().csd_ocm_age(self.handle, _stream_ptr(stream)), "csd_ocm_age")

    def merge(self, other: "Ocm", stream=None):
        """Add every pair of `other`, with its count, to this memory."""
        _check(lib().csd_ocm_merge(self.handle, other.handle, _stream_ptr(stream)), "csd_ocm_merge")

    def save(self, path: str, stream=None):
        """Write the memory to a file in the library's own format (csd_ocm_save): the table of Sec. 4.2 as it
        is handed from the calibration phase to deployment."""
        _check(lib().csd_ocm_save(self.handle, os.fsencode(path), _stream_ptr(stream)), "csd_ocm_save")

    @classmethod
    def load(cls, path: str, device: int = 0, n_slots: int = 0) -> "Ocm":
        """A new memory holding the pairs of a file written by `save` (n_slots = 0: as saved)."""
        if not torch.cuda.is_available():
            raise CsdError("a CUDA device is required")
        h = c_void_p()
        _check(lib().csd_ocm_load(byref(h), os.fsencode(path), n_slots, device), "csd_ocm_load")
        ocm = cls.__new__(cls)
        ocm.handle = h
        ocm.device = torch.device("cuda", device)
        ocm.n_slots = ocm.stats()["n_slots"]
        return ocm

    def stats(self, stream=None) -> dict:
        s = Stats()
        _check(lib().csd_ocm_stats(self.handle, byref(s), _stream_ptr(stream)), "csd_ocm_stats")
        return s.as_dict()


class StepBuffers:
    """Caller-owned device buffers of one step shape: outputs, optional diagnostics, workspace."""

    def __init__(self, B: int, K: int, V: int, dtype: torch.dtype, device="cuda", diag: bool = False):
        self.B, self.K, self.V = B, K, V
        self.dtype_code = CSD_F32 if dtype == torch.float32 else CSD_BF16
        dev = torch.device(device)
        self.accept_len = torch.empty(B, dtype=torch.int32, device=dev)
        self.next_token = torch.empty(B, dtype=torch.int32, device=dev)
        self.rescued_mask = torch.empty(B, K, dtype=torch.uint8, device=dev)
        self.rej_draft = torch.empty(B, K, dtype=torch.int32, device=dev)
        self.rej_target = torch.empty(B, K, dtype=torch.int32, device=dev)
        self.ws_bytes = csd_workspace_bytes(B, K, V, self.dtype_code)
        if self.ws_bytes == 0:
            raise CsdError(f"unsupported shape B={B} K={K} V={V}")
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        _check(lib().csd_workspace_init(_ptr(self.workspace), self.ws_bytes, _stream_ptr()), "csd_workspace_init")
        self.diag = None
        self._diag_struct = None
        if diag:
            f = dict(dtype=torch.float32, device=dev)
            self.diag = dict(
                m=torch.empty(B, K + 1, **f), s=torch.empty(B, K + 1, **f), lse=torch.empty(B, K + 1, **f),
                t=torch.empty(B, K + 1, dtype=torch.int32, device=dev),
                zd=torch.empty(B, K, **f), score=torch.empty(B, K, **f), p_d=torch.empty(B, K, **f),
                p_t=torch.empty(B, K, **f), cnt=torch.empty(B, K, dtype=torch.int32, device=dev))
            self._diag_struct = Diag(**{k: v.data_ptr() for k, v in self.diag.items()})


def _step_call(fn_name, logits, draft, ocm: Ocm, tau, buf: StepBuffers, stream):
    assert logits.is_cuda and draft.is_cuda and draft.dtype == torch.int32 and draft.is_contiguous()
    B, K1, V = logits.shape
    assert (B, K1 - 1, V) == (buf.B, buf.K, buf.V) and draft.shape == (B, K1 - 1)
    assert logits.stride(2) == 1 and _dtype_code(logits) == buf.dtype_code
    fn = getattr(lib(), fn_name)
    rc = fn(logits.data_ptr(), buf.dtype_code, B, K1 - 1, V, logits.stride(0), logits.stride(1),
            draft.data_ptr(), ocm.handle, c_float(tau),
            _ptr(buf.accept_len), _ptr(buf.next_token), _ptr(buf.rescued_mask), _ptr(buf.rej_draft), _ptr(buf.rej_target),
            byref(buf._diag_struct) if buf._diag_struct is not None else None,
            _ptr(buf.workspace), buf.ws_bytes, _stream_ptr(stream))
    _check(rc, fn_name)


def csd_verify(logits, draft, ocm: Ocm, tau: float, buf: StepBuffers, stream=None):
    """Verification loop of Algorithm 1 (greedy) for all rows; the memory is only read."""
    _step_call("csd_verify", logits, draft, ocm, tau, buf, stream)


def csd_step(logits, draft, ocm: Ocm, tau: float, buf: StepBuffers, stream=None):
    """csd_verify plus the memory update with the step's rejections, in one launch."""
    _step_call("csd_step", logits, draft, ocm, tau, buf, stream)


class HostStep:
    """csd_step_host: inputs and outputs in (pinned) host memory, copies inside the call."""

    def __init__(self, B, K, V, dtype: torch.dtype, device="cuda"):
        self.B, self.K, self.V = B, K, V
        self.dtype_code = CSD_F32 if dtype == torch.float32 else CSD_BF16
        self.bytes = csd_host_staging_bytes(B, K, V, self.dtype_code)
        self.staging = torch.empty(self.bytes, dtype=torch.uint8, device=device)
        assert self.staging.data_ptr() % 256 == 0
        self.accept_len = torch.empty(B, dtype=torch.int32).pin_memory()
        self.next_token = torch.empty(B, dtype=torch.int32).pin_memory()
        self.rescued_mask = torch.empty(B, K, dtype=torch.uint8).pin_memory()

    def __call__(self, logits_host: torch.Tensor, draft_host: torch.Tensor, ocm: Ocm, tau: float, stream=None):
        assert not logits_host.is_cuda and logits_host.is_contiguous() and draft_host.dtype == torch.int32
        assert tuple(logits_host.shape) == (self.B, self.K + 1, self.V) and _dtype_code(logits_host) == self.dtype_code
        rc = lib().csd_step_host(logits_host.data_ptr(), self.dtype_code, self.B, self.K, self.V,
                                 draft_host.data_ptr(), ocm.handle, c_float(tau),
                                 self.accept_len.data_ptr(), self.next_token.data_ptr(), self.rescued_mask.data_ptr(),
                                 self.staging.data_ptr(), self.bytes, _stream_ptr(stream))
        _check(rc, "csd_step_host")
        return self.accept_len, self.next_token, self.rescued_mask


STATIC_SCRATCH_BYTES = 1 << 20


def csd_verify_static(logits, draft, ocm: Ocm, tau: float, buf: StepBuffers, stream=None):
    """csd_verify with the scratch in the library's own fixed device array: for callers that
    cannot allocate device memory (buf.workspace is not used).  Calls must not overlap on the GPU."""
    assert logits.is_cuda and draft.is_cuda and draft.dtype == torch.int32 and draft.is_contiguous()
    B, K1, V = logits.shape
    assert (B, K1 - 1, V) == (buf.B, buf.K, buf.V) and logits.stride(2) == 1 and _dtype_code(logits) == buf.dtype_code
    rc = lib().csd_verify_static(
        logits.data_ptr(), buf.dtype_code, B, K1 - 1, V, logits.stride(0), logits.stride(1), draft.data_ptr(),
        ocm.handle, c_float(tau), _ptr(buf.accept_len), _ptr(buf.next_token), _ptr(buf.rescued_mask),
        _ptr(buf.rej_draft), _ptr(buf.rej_target),
        byref(buf._diag_struct) if buf._diag_struct is not None else None, _stream_ptr(stream))
    _check(rc, "csd_verify_static")


class SampledBuffers:
    """Caller-owned device buffers of one stochastic step shape: outputs, diagnostics, workspace."""

    def __init__(self, B: int, K: int, V: int, dtype: torch.dtype, device="cuda", diag: bool = True):
        self.B, self.K, self.V = B, K, V
        self.dtype_code = CSD_F32 if dtype == torch.float32 else CSD_BF16
        dev = torch.device(device)
        i32 = dict(dtype=torch.int32, device=dev)
        self.accept_len = torch.empty(B, **i32)
        self.next_token = torch.empty(B, **i32)
        self.rescued_mask = torch.empty(B, K, dtype=torch.uint8, device=dev)
        self.rej_draft = torch.empty(B, K, **i32)
        self.rej_target = torch.empty(B, K, **i32)
        self.ws_bytes = int(lib().csd_sampled_workspace_bytes(B, K, V, self.dtype_code))
        if self.ws_bytes == 0:
            raise CsdError(f"unsupported shape B={B} K={K} V={V}")
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self.diag = None
        self._diag_struct = None
        if diag:
            f = dict(dtype=torch.float32, device=dev)
            self.diag = dict(alpha=torch.empty(B, K, **f), accepted=torch.empty(B, K, dtype=torch.uint8, device=dev),
                             t_star=torch.empty(B, K, **i32), lse_p=torch.empty(B, K + 1, **f), lse_q=torch.empty(B, K, **f),
                             score=torch.empty(B, K, **f), cnt=torch.empty(B, K, **i32), bonus=torch.empty(B, **i32))
            self._diag_struct = SampledDiag(**{k: v.data_ptr() for k, v in self.diag.items()})


def _sampled_call(fn_name, logits, draft_logits, draft, r_accept, seed, temperature, ocm: Ocm, tau, buf, stream):
    assert logits.is_cuda and draft_logits.is_cuda and draft.is_cuda and r_accept.is_cuda
    assert draft.dtype == torch.int32 and draft.is_contiguous() and r_accept.dtype == torch.float32 and r_accept.is_contiguous()
    B, K1, V = logits.shape
    assert (B, K1 - 1, V) == (buf.B, buf.K, buf.V) and tuple(draft_logits.shape) == (B, K1 - 1, V)
    assert logits.stride(2) == 1 and draft_logits.stride(2) == 1 and draft_logits.dtype == logits.dtype
    assert _dtype_code(logits) == buf.dtype_code and tuple(draft.shape) == (B, K1 - 1) == tuple(r_accept.shape)
    rc = getattr(lib(), fn_name)(
        logits.data_ptr(), draft_logits.data_ptr(), buf.dtype_code, B, K1 - 1, V, logits.stride(0), logits.stride(1),
        draft_logits.stride(0), draft_logits.stride(1), draft.data_ptr(), r_accept.data_ptr(), c_uint64(seed),
        c_float(temperature), ocm.handle, c_float(tau), _ptr(buf.accept_len), _ptr(buf.next_token),
        _ptr(buf.rescued_mask), _ptr(buf.rej_draft), _ptr(buf.rej_target),
        byref(buf._diag_struct) if buf._diag_struct is not None else None, _ptr(buf.workspace), buf.ws_bytes,
        _stream_ptr(stream))
    _check(rc, fn_name)


def csd_verify_sampled(logits, draft_logits, draft, r_accept, seed: int, temperature: float, ocm: Ocm, tau: float,
                       buf: SampledBuffers, stream=None):
    """Algorithm 1 at temperature T > 0 (stochastic acceptance, residual draws); the memory is only read."""
    _sampled_call("csd_verify_sampled", logits, draft_logits, draft, r_accept, seed, temperature, ocm, tau, buf, stream)


def csd_step_sampled(logits, draft_logits, draft, r_accept, seed: int, temperature: float, ocm: Ocm, tau: float,
                     buf: SampledBuffers, stream=None):
    """csd_verify_sampled followed by the memory update with the step's recorded pairs."""
    _sampled_call("csd_step_sampled", logits, draft_logits, draft, r_accept, seed, temperature, ocm, tau, buf, stream)


def sampled_launches_per_step(B: int, K: int, V: int, dtype) -> int:
    """Kernel launches one csd_step_sampled call of this shape makes (for launch counts in reports)."""
    return int(lib().csd_sampled_launches(B, K, V, CSD_BF16 if dtype == torch.bfloat16 else CSD_F32))


def csd_sampled_set_rounds(mode: int = 0):
    """0 automatic, 1 every draw in one round, 2 two rounds of draws on demand."""
    _check(lib().csd_sampled_set_rounds(mode), "csd_sampled_set_rounds")


class LmheadBuffers(StepBuffers):
    """Outputs, optional diagnostics and workspace of the step that starts from the LM head's inputs."""

    def __init__(self, B: int, K: int, H: int, V: int, device="cuda", diag: bool = False):
        self.H = H
        bytes_ = int(lib().csd_lmhead_workspace_bytes(B, K, H, V))
        if bytes_ == 0:
            raise CsdError(f"unsupported shape B={B} K={K} H={H} V={V} (H % 64 == 0 is required)")
        super().__init__(B, K, V, torch.bfloat16, device=device, diag=diag)
        self.ws_bytes = bytes_
        self.workspace = torch.empty(bytes_, dtype=torch.uint8, device=torch.device(device))


def csd_lmhead_shape(B, K, H, V):
    g, n, t, per = c_int(), c_int(), c_int(), c_int()
    _check(lib().csd_lmhead_shape(B, K, H, V, byref(g), byref(n), byref(t), byref(per)), "csd_lmhead_shape")
    pairs = bool(lib().csd_lmhead_uses_pairs(B, K))
    return dict(grid=g.value, tile_cols=n.value, tiles=t.value, tiles_per_block=per.value,
                kernel="lmhead_stats_pair_kernel" if pairs else "lmhead_stats_kernel")


def _lmhead_call(fn_name, hidden, weight, draft, ocm: Ocm, tau, buf: LmheadBuffers, stream):
    assert hidden.is_cuda and weight.is_cuda and draft.is_cuda and draft.dtype == torch.int32 and draft.is_contiguous()
    assert hidden.dtype == torch.bfloat16 and weight.dtype == torch.bfloat16 and hidden.is_contiguous() and weight.is_contiguous()
    B, K1, H = hidden.shape
    V, H2 = weight.shape
    assert (B, K1 - 1, H, V) == (buf.B, buf.K, buf.H, buf.V) and H2 == H and tuple(draft.shape) == (B, K1 - 1)
    rc = getattr(lib(), fn_name)(hidden.data_ptr(), weight.data_ptr(), B, K1 - 1, H, V, draft.data_ptr(), ocm.handle, c_float(tau),
                                 _ptr(buf.accept_len), _ptr(buf.next_token), _ptr(buf.rescued_mask), _ptr(buf.rej_draft),
                                 _ptr(buf.rej_target), byref(buf._diag_struct) if buf._diag_struct is not None else None,
                                 _ptr(buf.workspace), buf.ws_bytes, _stream_ptr(stream))
    _check(rc, fn_name)


def csd_verify_lmhead(hidden, weight, draft, ocm: Ocm, tau: float, buf: LmheadBuffers, stream=None):
    """csd_verify on the logits hidden @ weight^T, which are never stored; the memory is only read."""
    _lmhead_call("csd_verify_lmhead", hidden, weight, draft, ocm, tau, buf, stream)


def csd_step_lmhead(hidden, weight, draft, ocm: Ocm, tau: float, buf: LmheadBuffers, stream=None):
    """csd_step on the logits hidden @ weight^T, which are never stored."""
    _lmhead_call("csd_step_lmhead", hidden, weight, draft, ocm, tau, buf, stream)


class EarlyExitBuffers(StepBuffers):
    """Outputs, optional diagnostics and workspace of csd_step_early_exit for one shape and first-phase length."""

    def __init__(self, B: int, K: int, V: int, dtype: torch.dtype, first: int = 0, device="cuda", diag: bool = False):
        super().__init__(B, K, V, dtype, device=device, diag=diag)
        self.first = first
        self.ws_bytes = int(lib().csd_early_exit_workspace_bytes(B, K, V, self.dtype_code, first))
        if self.ws_bytes == 0:
            raise CsdError(f"unsupported shape for the two-phase step: B={B} K={K} V={V}")
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=torch.device(device))


def csd_step_early_exit(logits, draft, ocm: Ocm, tau: float, buf: EarlyExitBuffers, stream=None):
    """csd_step in two phases: batch rows that stop within the first phase are not read any further."""
    assert logits.is_cuda and draft.is_cuda and draft.dtype == torch.int32 and draft.is_contiguous()
    B, K1, V = logits.shape
    assert (B, K1 - 1, V) == (buf.B, buf.K, buf.V) and logits.stride(2) == 1 and _dtype_code(logits) == buf.dtype_code
    rc = lib().csd_step_early_exit(
        logits.data_ptr(), buf.dtype_code, B, K1 - 1, V, logits.stride(0), logits.stride(1), draft.data_ptr(), ocm.handle,
        c_float(tau), buf.first, _ptr(buf.accept_len), _ptr(buf.next_token), _ptr(buf.rescued_mask), _ptr(buf.rej_draft),
        _ptr(buf.rej_target), byref(buf._diag_struct) if buf._diag_struct is not None else None, _ptr(buf.workspace),
        buf.ws_bytes, _stream_ptr(stream))
    _check(rc, "csd_step_early_exit")


def csd_lmhead_set_tuning(kblocks_per_stage: int = 0, mma_cols: int = 0):
    _check(lib().csd_lmhead_set_tuning(kblocks_per_stage, mma_cols), "csd_lmhead_set_tuning")


def csd_lmhead_set_pairing(mode: int = 0):
    """0 automatic, 1 one block per SM, 2 pairs of blocks (clusters of two)."""
    _check(lib().csd_lmhead_set_pairing(mode), "csd_lmhead_set_pairing")
