"""Seeded synthetic inputs shaped like the paper's workloads.

This module only *makes inputs* (logits, draft tokens, rejection-pair streams);
it holds none of the method's arithmetic and is the one module that both the
CUDA path's tests and the CPU oracle's tests draw from.

The logits stand in for target-model logits of the Llama-3 (V = 128256) and
Qwen-2.5 (V = 151936 / 152064) vocabularies of Sec. 5.1:

  * every logit is N(0, sigma^2) noise; one seeded "target top" token per row is
    raised by `peak` (a constant, or U(lo, hi) drawn once per batch row);
  * each draft position is one of three kinds, drawn with the workload's mix:
      match    the draft equals the row's true arg-max (lowest index on ties),
      synonym  a (target, draft) pair is drawn from a fixed seeded map with
               Zipf(a) rank weights; the target becomes the raised token and the
               draft's logit is set to  z[target] - U(0, 3), so the ratio of
               Eq. 3 is e^-U in (0.05, 1]  (the spread of Observation 2);
      uniform  the draft is uniform on [0, V);
    the skewed map stands in for Observation 1 (few pairs make most rejections);
  * values are made in fp32 and rounded to bf16 (RNE) where the workload says so.

Every step is regenerable from (seed, workload id, step index).
"""

from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    wid: int
    B: int
    K: int
    V: int
    dtype: str                      # "f32" | "bf16"
    sigma: float
    peak: tuple                     # (lo, hi); lo == hi for a constant peak
    mix: tuple                      # (match, synonym, uniform) probabilities
    n_pairs: int
    zipf_a: float
    ocm_slots: int
    taus: tuple
    steps: int
    prewarm: tuple = ("none", 0)    # ("steps", n) | ("pairs", n) | ("none", 0)
    lam: int = 6
    checkpoint_every: int = 0
    notes: str = ""

    @property
    def rows(self) -> int:
        return self.B * (self.K + 1)

    @property
    def elt_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def logit_bytes(self) -> int:
        return self.rows * self.V * self.elt_bytes

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


WORKLOADS = {
    "tiny": Workload("tiny", 1, B=1, K=4, V=32000, dtype="f32", sigma=1.0, peak=(8.0, 8.0),
                     mix=(0.60, 0.25, 0.15), n_pairs=500, zipf_a=1.1, ocm_slots=4096,
                     taus=(0.3,), steps=1000),
    "single_stream": Workload("single_stream", 2, B=1, K=8, V=128256, dtype="bf16", sigma=1.0,
                              peak=(8.0, 8.0), mix=(0.60, 0.25, 0.15), n_pairs=2000, zipf_a=1.1,
                              ocm_slots=65536, taus=(0.1, 0.3, 0.5), steps=10000,
                              prewarm=("steps", 5000)),
    "batched_serving": Workload("batched_serving", 3, B=32, K=5, V=151936, dtype="bf16", sigma=1.0,
                                peak=(4.0, 10.0), mix=(0.50, 0.30, 0.20), n_pairs=5000, zipf_a=1.1,
                                ocm_slots=262144, taus=(0.3,), steps=5000),
    "large_batch": Workload("large_batch", 4, B=128, K=8, V=128256, dtype="f32", sigma=1.5,
                            peak=(6.0, 6.0), mix=(0.55, 0.30, 0.15), n_pairs=5000, zipf_a=1.1,
                            ocm_slots=1048576, taus=(0.2, 0.4), steps=1000,
                            prewarm=("pairs", 200000)),
    "ocm_contention": Workload("ocm_contention", 5, B=64, K=6, V=152064, dtype="bf16", sigma=1.0,
                               peak=(8.0, 8.0), mix=(0.30, 0.50, 0.20), n_pairs=256, zipf_a=1.5,
                               ocm_slots=65536, taus=(0.3,), steps=100000, checkpoint_every=10000),
}


def _seed(seed: int, wid: int, stream: int, step: int) -> int:
    x = (seed * 1000003 + wid * 7919 + stream * 15485863 + step * 104729 + 12345) % (2**62)
    return int(x)


class Synth:
    """Generator of one workload's step inputs on `device` ("cpu" or "cuda")."""

    def __init__(self, wl: Workload, seed: int = 0, device="cpu"):
        self.wl = wl
        self.seed = int(seed)
        self.device = torch.device(device)
        g = torch.Generator(device="cpu")
        g.manual_seed(_seed(self.seed, wl.wid, 1, 0))
        # the synonym map: n_pairs (target, draft) token pairs with distinct members
        tgt = torch.randint(0, wl.V, (wl.n_pairs,), generator=g)
        off = torch.randint(1, wl.V, (wl.n_pairs,), generator=g)
        drf = (tgt + off) % wl.V
        self.map_target = tgt.to(self.device)
        self.map_draft = drf.to(self.device)
        rank = torch.arange(1, wl.n_pairs + 1, dtype=torch.float64)
        w = rank.pow(-wl.zipf_a)
        self.pair_cdf = (torch.cumsum(w, 0) / w.sum()).to(torch.float32).to(self.device)

    def _gen(self, stream: int, step: int) -> torch.Generator:
        g = torch.Generator(device=self.device)
        g.manual_seed(_seed(self.seed, self.wl.wid, stream, step))
        return g

    def _draw_pairs(self, u: torch.Tensor) -> torch.Tensor:
        idx = torch.searchsorted(self.pair_cdf, u.contiguous())
        return idx.clamp_(max=self.wl.n_pairs - 1)

    def prewarm_pairs(self, n: int):
        """n (draft, target) rejection pairs drawn from the Zipf map, int32 each."""
        g = self._gen(3, 0)
        u = torch.rand(n, generator=g, device=self.device)
        idx = self._draw_pairs(u)
        return self.map_draft[idx].to(torch.int32), self.map_target[idx].to(torch.int32)

    def step(self, step: int):
        """(logits[B, K+1, V] in the workload dtype, draft[B, K] int32) for one step."""
        wl, dev = self.wl, self.device
        B, K, V = wl.B, wl.K, wl.V
        g = self._gen(2, step)
        z = torch.randn(B, K + 1, V, generator=g, device=dev, dtype=torch.float32)
        if wl.sigma != 1.0:
            z.mul_(wl.sigma)
        kind_u = torch.rand(B, K, generator=g, device=dev)
        pair_u = torch.rand(B, K, generator=g, device=dev)
        gap_u = torch.rand(B, K, generator=g, device=dev)
        peak_u = torch.rand(B, generator=g, device=dev)
        top = torch.randint(0, V, (B, K + 1), generator=g, device=dev)
        uni = torch.randint(0, V, (B, K), generator=g, device=dev)

        is_match = kind_u < wl.mix[0]
        is_syn = (~is_match) & (kind_u < wl.mix[0] + wl.mix[1])
        pair = self._draw_pairs(pair_u.reshape(-1)).reshape(B, K)
        syn_t = self.map_target[pair]
        syn_d = self.map_draft[pair]
        top[:, :K] = torch.where(is_syn, syn_t, top[:, :K])

        peak = wl.peak[0] + (wl.peak[1] - wl.peak[0]) * peak_u          # per batch row
        z.scatter_add_(2, top.unsqueeze(-1), peak.view(B, 1, 1).expand(B, K + 1, 1).contiguous())
        # synonym positions: the draft's logit sits U(0, 3) below the raised token
        zt = z[:, :K].gather(2, top[:, :K].unsqueeze(-1)).squeeze(-1)
        old = z[:, :K].gather(2, syn_d.unsqueeze(-1)).squeeze(-1)
        new = torch.where(is_syn, zt - 3.0 * gap_u, old)
        z[:, :K].scatter_(2, syn_d.unsqueeze(-1), new.unsqueeze(-1))

        z = z.to(wl.torch_dtype)

        # the row's true arg-max, lowest index on ties (chunked to bound memory)
        arg = torch.empty(B, K, dtype=torch.int64, device=dev)
        ar = torch.arange(V, device=dev, dtype=torch.int32)
        big = torch.tensor(V, device=dev, dtype=torch.int32)
        cb = max(1, (1 << 24) // (K * V))
        for b0 in range(0, B, cb):
            zz = z[b0:b0 + cb, :K]
            mx = zz.amax(dim=2, keepdim=True)
            arg[b0:b0 + cb] = torch.where(zz == mx, ar, big).amin(dim=2).to(torch.int64)
        draft = torch.where(is_match, arg, torch.where(is_syn, syn_d, uni)).to(torch.int32)
        return z.contiguous(), draft.contiguous()


    def step_sampled(self, step: int, draft_noise: float = 0.3, draft_margin: float = 1.0):
        """Inputs of one STOCHASTIC step: (logits, draft_logits[B, K, V], draft, r[B, K] float32).

        The target logits and draft tokens are those of `step`.  The draft model's logits are
        the target's plus N(0, draft_noise^2) (a drafter that mostly agrees), except that at
        every position the drafter's favourite is its own draft token: that logit is raised
        to the row's maximum plus `draft_margin`.  r is uniform on [0, 1).
        """
        wl, dev = self.wl, self.device
        z, draft = self.step(step)
        g = self._gen(4, step)
        y = z[:, :wl.K].to(torch.float32).clone()
        y.add_(torch.randn(y.shape, generator=g, device=dev, dtype=torch.float32), alpha=draft_noise)
        top = y.amax(dim=2, keepdim=True) + draft_margin
        y.scatter_(2, draft.to(torch.int64).unsqueeze(-1), top)
        r = torch.rand(wl.B, wl.K, generator=g, device=dev, dtype=torch.float32)
        return z, y.to(wl.torch_dtype).contiguous(), draft, r.contiguous()


    # ---- inputs of the LM head: the step that never stores its logits --------------------------------
    def lmhead_weight(self, H: int) -> torch.Tensor:
        """W[V, H] bf16, N(0, 1/H) entries: with hidden rows of N(0, sigma^2) entries the logits hidden . W[v]
        are N(0, sigma^2) noise, as in `step`.  Fixed by (seed, workload)."""
        g = self._gen(5, 0)
        w = torch.randn(self.wl.V, H, generator=g, device=self.device, dtype=torch.float32)
        return w.mul_(H ** -0.5).to(torch.bfloat16).contiguous()

    def step_lmhead(self, step: int, W: torch.Tensor):
        """(hidden[B, K+1, H] bf16, draft[B, K] int32) for one step whose logits are hidden @ W^T.

        The same recipe as `step`, expressed through the hidden state: a row is noise plus `peak` times the
        (normalised) weight row of its raised token, which lifts that token's logit by `peak`; at a synonym
        position a component along the draft token's weight row puts its logit U(0, 3) below the raised
        token's (up to the small overlap of two random weight rows).  "Match" drafts are the arg-max of the
        finished row, taken from a float32 product of the rounded inputs."""
        wl, dev = self.wl, self.device
        B, K, V = wl.B, wl.K, wl.V
        H = W.shape[1]
        g = self._gen(6, step)
        h = torch.randn(B, K + 1, H, generator=g, device=dev, dtype=torch.float32).mul_(wl.sigma)
        kind_u = torch.rand(B, K, generator=g, device=dev)
        pair_u = torch.rand(B, K, generator=g, device=dev)
        gap_u = torch.rand(B, K, generator=g, device=dev)
        peak_u = torch.rand(B, generator=g, device=dev)
        top = torch.randint(0, V, (B, K + 1), generator=g, device=dev)
        uni = torch.randint(0, V, (B, K), generator=g, device=dev)
        is_match = kind_u < wl.mix[0]
        is_syn = (~is_match) & (kind_u < wl.mix[0] + wl.mix[1])
        pair = self._draw_pairs(pair_u.reshape(-1)).reshape(B, K)
        syn_t, syn_d = self.map_target[pair], self.map_draft[pair]
        top[:, :K] = torch.where(is_syn, syn_t, top[:, :K])
        peak = (wl.peak[0] + (wl.peak[1] - wl.peak[0]) * peak_u).view(B, 1, 1)
        wt = W[top].to(torch.float32)                                        # [B, K+1, H]
        h = h + peak * wt / wt.pow(2).sum(-1, keepdim=True)
        wd = W[syn_d].to(torch.float32)                                      # [B, K, H]
        z_top = (h[:, :K] * wt[:, :K]).sum(-1)
        z_d = (h[:, :K] * wd).sum(-1)
        lift = torch.where(is_syn, z_top - 3.0 * gap_u - z_d, torch.zeros_like(z_d))
        h[:, :K] = h[:, :K] + lift.unsqueeze(-1) * wd / wd.pow(2).sum(-1, keepdim=True)
        h = h.to(torch.bfloat16).contiguous()
        arg = torch.empty(B, K, dtype=torch.int64, device=dev)
        for b in range(B):                                                   # a [K, V] product at a time
            arg[b] = (h[b, :K].to(torch.float32) @ W.to(torch.float32).T if V * H <= (1 << 24) else
                      torch.cat([h[b, :K].to(torch.float32) @ W[v0:v0 + 32768].to(torch.float32).T
                                 for v0 in range(0, V, 32768)], dim=1)).argmax(dim=1)
        draft = torch.where(is_match, arg, torch.where(is_syn, syn_d, uni)).to(torch.int32)
        return h, draft.contiguous()


def logits_to_numpy(z: torch.Tensor):
    """Exact host copy for the oracle: float32 array (bf16 widens exactly)."""
    return z.detach().to("cpu").to(torch.float32).numpy()


def logits_bits_numpy(z: torch.Tensor):
    """(array, is_bf16_bits): float32 values, or the raw 16-bit patterns of a bf16 tensor."""
    z = z.detach().to("cpu").contiguous()
    if z.dtype == torch.bfloat16:
        return z.view(torch.int16).numpy().view("uint16"), True
    return z.numpy(), False
