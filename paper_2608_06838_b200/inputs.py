"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the method itself: it only draws random
tensors.  Both the CUDA tests/benchmarks and the CPU oracle tests take their
inputs from here, so the two sides always see identical bits.

Recipe (one linear-recurrence layer, micro-batch 1 as in the paper's setup,
Section 4.1; heads and state width follow its 3B-32B models):
  q, k : N(0,1) rows, either divided by sqrt(d_k) ("scaled") or L2-normalised
         per (token, head) ("l2"), then rounded to the storage dtype
  v, dO: N(0,1)
  g    : -softplus(N(0,1)) * g_scale  (log-decay per token per head, fp32)
  S_in, dS_out : N(0, sigma) element-wise fp32, or absent
Each tensor has its own generator stream (seed * 16 + tensor id), so a tensor
does not change when another one is added or resized.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch


@dataclass
class Workload:
    name: str
    B: int
    H: int
    d_k: int
    d_v: int
    seg_lens: List[int]
    chunk: int
    dtype: str = "bf16"            # storage type of q,k,v,o,dO,dq,dk,dv: "bf16" or "f32"
    qk_norm: str = "l2"            # "l2" or "scaled"
    g_scale: float = 1.0
    s_in_sigma: Optional[float] = None      # None = no incoming state (S_0 = 0)
    ds_out_sigma: Optional[float] = None    # None = no incoming state gradient
    seed: int = 0

    @property
    def T(self) -> int:
        return int(sum(self.seg_lens))


def configs() -> List[Workload]:
    """The five benchmark configurations (index = configuration number - 1)."""
    return [
        Workload("tiny", 1, 2, 32, 32, [128, 128], 32, dtype="f32", qk_norm="scaled"),
        Workload("32k", 1, 16, 128, 128, [4096] * 8, 64),
        Workload("64k-nonuniform", 1, 32, 128, 128,
                 [12288, 10240, 8192, 8192, 8192, 6144, 6144, 6144], 64, s_in_sigma=0.02),
        Workload("256k", 1, 32, 128, 128, [16384] * 16, 64, ds_out_sigma=0.02),
        Workload("128k-sweep", 1, 40, 128, 128, [4096] * 32, 64),
    ]


def sweep_config(seg_len: int) -> Workload:
    """Configuration 5 with a given uniform segment length."""
    T = 131072
    return Workload("128k-seg%d" % seg_len, 1, 40, 128, 128, [seg_len] * (T // seg_len), 64)


def _gen(device, seed: int, tid: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed * 16 + tid)
    return g


def make_inputs(w: Workload, device="cpu"):
    """Returns a dict of tensors: q,k [B,T,H,d_k]; v,dO [B,T,H,d_v] in the storage dtype;
    g [B,T,H] fp32; S_in, dS_out [B,H,d_k,d_v] fp32 or None."""
    dev = torch.device(device)
    st = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    B, T, H = w.B, w.T, w.H

    def randn(tid, *shape):
        return torch.randn(*shape, generator=_gen(dev, w.seed, tid), device=dev, dtype=torch.float32)

    def qk(tid):
        x = randn(tid, B, T, H, w.d_k)
        if w.qk_norm == "l2":
            x = x / x.norm(dim=-1, keepdim=True)
        else:
            x = x / (w.d_k ** 0.5)
        return x.to(st)

    out = {
        "q": qk(0),
        "k": qk(1),
        "v": randn(2, B, T, H, w.d_v).to(st),
        "g": -torch.nn.functional.softplus(randn(3, B, T, H)) * w.g_scale,
        "dO": randn(4, B, T, H, w.d_v).to(st),
        "S_in": None,
        "dS_out": None,
    }
    if w.s_in_sigma is not None:
        out["S_in"] = randn(5, B, H, w.d_k, w.d_v) * w.s_in_sigma
    if w.ds_out_sigma is not None:
        out["dS_out"] = randn(6, B, H, w.d_k, w.d_v) * w.ds_out_sigma
    return out


def make_variant_inputs(w: Workload, device="cpu", conv_width: int = 4):
    """make_inputs plus what the extension operators take:
      g_channel [B,T,H,d_k] : -softplus(N(0,1)) * g_scale, one log-decay per key channel (diagonal family)
      beta [B,T,H]          : sigmoid(N(0,1)), the write strength of the delta rule
      conv_x, conv_dy [B,T,C], conv_w [W,C] / sqrt(W), conv_tail, conv_dtail [B,W-1,C] with C = H*d_v: N(0,1)"""
    out = make_inputs(w, device)
    dev = torch.device(device)
    B, T, H = w.B, w.T, w.H
    C = H * w.d_v

    def randn(tid, *shape):
        return torch.randn(*shape, generator=_gen(dev, w.seed, tid), device=dev, dtype=torch.float32)

    out["g_channel"] = -torch.nn.functional.softplus(randn(7, B, T, H, w.d_k)) * w.g_scale
    out["beta"] = torch.sigmoid(randn(8, B, T, H))
    out["conv_x"] = randn(9, B, T, C)
    out["conv_dy"] = randn(10, B, T, C)
    out["conv_w"] = randn(11, conv_width, C) / (conv_width ** 0.5)
    out["conv_tail"] = randn(12, B, max(conv_width - 1, 0), C)
    out["conv_dtail"] = randn(13, B, max(conv_width - 1, 0), C)
    return out


def to_f64(t):
    """Widen a tensor (or None) to a float64 numpy array on the host - the exact values the GPU sees."""
    return None if t is None else t.detach().to("cpu", torch.float64).numpy()
