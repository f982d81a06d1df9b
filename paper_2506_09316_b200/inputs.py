"""Seeded synthetic inputs for the dual-state linear attention (DSLA) layer.

This module only draws random numbers and shapes them; it holds none of the
layer's arithmetic.  Both the CUDA parity tests and the CPU checker are fed from
here so that they see bit-identical arrays.

Draw order (fixed, so a seed names one data set): q, k, v, g_hist, g_rec, gamma.
  q, k, v   ~ N(0, 1) / sqrt(d), rounded to the working dtype (fp32 or bf16)
  g_hist    = logistic(N(6, 0.5))   per (token, head)   ~ 0.9975 (slow decay)
  g_rec     = logistic(N(1, 0.5))   per (token, head)   ~ 0.73   (fast decay)
  gamma     ~ U(0, 1)               per head
Layouts: q, k, v are [T_total, H, d] (token-major, d contiguous); gates are
[T_total, H] fp32; cu_seqlens is int32 [N + 1].
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch


def _logistic(x):
    return 1.0 / (1.0 + np.exp(-x))


@dataclass
class DslaInputs:
    q: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    g_hist: torch.Tensor
    g_rec: torch.Tensor
    gamma: torch.Tensor
    cu_seqlens: torch.Tensor  # int32 [N+1]
    H: int
    d: int
    dtype: torch.dtype
    seed: int
    extra: dict = field(default_factory=dict)

    @property
    def N(self) -> int:
        return self.cu_seqlens.numel() - 1

    @property
    def T_total(self) -> int:
        return int(self.q.shape[0])

    @property
    def seqlens(self):
        c = self.cu_seqlens.cpu().numpy()
        return (c[1:] - c[:-1]).tolist()

    def to(self, device):
        kw = dict(q=self.q.to(device), k=self.k.to(device), v=self.v.to(device),
                  g_hist=self.g_hist.to(device), g_rec=self.g_rec.to(device),
                  gamma=self.gamma.to(device), cu_seqlens=self.cu_seqlens.to(device))
        return DslaInputs(H=self.H, d=self.d, dtype=self.dtype, seed=self.seed, extra=self.extra, **kw)

    def as_f64(self):
        """Exact widening of every array to numpy float64 (bf16 -> fp64 is exact)."""
        f = lambda t: t.detach().cpu().to(torch.float64).numpy()
        return dict(q=f(self.q), k=f(self.k), v=f(self.v), g_hist=f(self.g_hist), g_rec=f(self.g_rec),
                    gamma=f(self.gamma), cu_seqlens=self.cu_seqlens.cpu().numpy().astype(np.int32))


def make_packed(seed: int, seqlens, H: int, d: int, dtype=torch.float32,
                hist_mu: float = 6.0, rec_mu: float = 1.0, gate_sigma: float = 0.5) -> DslaInputs:
    """Packed (varlen) inputs drawn on the host with numpy's PCG64."""
    seqlens = [int(x) for x in seqlens]
    T = int(sum(seqlens))
    rng = np.random.default_rng(seed)
    s = 1.0 / math.sqrt(d)
    q = (rng.standard_normal((T, H, d), dtype=np.float32) * s).astype(np.float32)
    k = (rng.standard_normal((T, H, d), dtype=np.float32) * s).astype(np.float32)
    v = (rng.standard_normal((T, H, d), dtype=np.float32) * s).astype(np.float32)
    g_hist = _logistic(rng.normal(hist_mu, gate_sigma, (T, H))).astype(np.float32)
    g_rec = _logistic(rng.normal(rec_mu, gate_sigma, (T, H))).astype(np.float32)
    gamma = rng.uniform(0.0, 1.0, (H,)).astype(np.float32)
    cu = np.zeros(len(seqlens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(seqlens)
    tt = lambda a: torch.from_numpy(a).to(dtype)
    return DslaInputs(q=tt(q), k=tt(k), v=tt(v), g_hist=torch.from_numpy(g_hist), g_rec=torch.from_numpy(g_rec),
                      gamma=torch.from_numpy(gamma), cu_seqlens=torch.from_numpy(cu), H=H, d=d, dtype=dtype, seed=seed)


def make_dense(seed: int, B: int, T: int, H: int, d: int, dtype=torch.float32, **kw) -> DslaInputs:
    return make_packed(seed, [T] * B, H, d, dtype, **kw)


def make_packed_device(seed: int, seqlens, H: int, d: int, dtype=torch.bfloat16, device="cuda",
                       hist_mu: float = 6.0, rec_mu: float = 1.0, gate_sigma: float = 0.5) -> DslaInputs:
    """Same distributions drawn on the device (for workloads too large to draw on the host).

    The stream differs from make_packed's; parity checks on such inputs copy the
    slices they need back to the host, so both sides still see identical values.
    """
    seqlens = [int(x) for x in seqlens]
    T = int(sum(seqlens))
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    s = 1.0 / math.sqrt(d)

    def normal(shape, scale):
        # drawn in pieces so no fp32 temporary larger than ~1 GiB is held
        out = torch.empty(shape, dtype=dtype, device=device)
        rows = max(1, (1 << 28) // max(1, int(np.prod(shape[1:]))))
        for r0 in range(0, shape[0], rows):
            r1 = min(shape[0], r0 + rows)
            out[r0:r1] = (torch.randn((r1 - r0,) + tuple(shape[1:]), generator=g, device=device,
                                      dtype=torch.float32) * scale).to(dtype)
        return out

    q = normal((T, H, d), s)
    k = normal((T, H, d), s)
    v = normal((T, H, d), s)
    g_hist = torch.sigmoid(torch.randn((T, H), generator=g, device=device) * gate_sigma + hist_mu)
    g_rec = torch.sigmoid(torch.randn((T, H), generator=g, device=device) * gate_sigma + rec_mu)
    gamma = torch.rand((H,), generator=g, device=device)
    cu = np.zeros(len(seqlens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(seqlens)
    return DslaInputs(q=q, k=k, v=v, g_hist=g_hist, g_rec=g_rec, gamma=gamma,
                      cu_seqlens=torch.from_numpy(cu).to(device), H=H, d=d, dtype=dtype, seed=seed)


def make_states(seed: int, num_slots: int, H: int, d_k: int, d_v: int, std: float = 0.02, device="cpu"):
    """Dual states [num_slots, 2, H, d_k, d_v] fp32 ~ N(0, std); index 0 = history, 1 = recency."""
    if device == "cpu":
        rng = np.random.default_rng(seed)
        return torch.from_numpy((rng.standard_normal((num_slots, 2, H, d_k, d_v), dtype=np.float32) * std))
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    out = torch.empty((num_slots, 2, H, d_k, d_v), dtype=torch.float32, device=device)
    for s0 in range(num_slots):
        out[s0] = torch.randn((2, H, d_k, d_v), generator=g, device=device) * std
    return out


def ragged_lengths(seed: int, n: int = 64, lo: int = 1024, hi: int = 65536):
    """n prompt lengths, log-uniform in [lo, hi] (the serving-mix recipe)."""
    rng = np.random.default_rng(seed)
    return np.rint(np.exp(rng.uniform(math.log(lo), math.log(hi), n))).astype(np.int64).tolist()


# The five named workloads (shapes and seeds); tensors are drawn by the callers.
CONFIGS = {
    "cfg1": dict(seed=1001, B=1, H=4, d=64, T=512, decode_steps=64, dtype="f32"),
    "cfg2": dict(seed=1002, B=1, H=32, d=128, T=4096, dtype="bf16", chunk=64),
    "cfg3": dict(seed=1003, B=1, H=32, d=128, T=65536, dtype="bf16", chunk=64),
    "cfg4": dict(seed=1004, B=128, H=32, d=128, layers=32, steps=256, ring=8, dtype="bf16", state_std=0.02),
    "cfg5": dict(seed=1005, N=64, H=32, d=128, lo=1024, hi=65536, decode_steps=128, dtype="bf16"),
}
