"""Seeded synthetic inputs and the named workload shapes.

This module holds no arithmetic of the attention method: it draws random tensors with
the shapes and value distributions of the paper's layers (Table 1 head size 128; the
qk-norm of the paper's models is stood in for by dividing every q and k row by its RMS)
and hands the same bits to both the CUDA path and the CPU checker.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H_q: int
    H_kv: int
    T: int
    d: int
    w: int
    dtype: str            # "bf16" or "f32" (I/O type; accumulation is always fp32)
    seed: int
    qk_rms_norm: bool     # divide every q, k row by its RMS (qk-norm stand-in)
    q_prescale: float     # multiply q by this on the host (config 1 folds 1/sqrt(d) into q)
    scale: float          # logit scale handed to the operator (SWA logits only)
    decode_steps: int = 0

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five named configurations (shapes of the paper's 3B / 12B layers, synthetic data).
C1 = Workload("c1_fp32_small", 1, 2, 2, 1024, 64, 128, "f32", 1001, False, 1.0 / 8.0, 1.0)
C2 = Workload("c2_3b_fwd", 4, 16, 16, 4096, 128, 512, "bf16", 1002, True, 1.0,
              1.0 / math.sqrt(128.0))
C3 = Workload("c3_12b_gqa_fwd", 2, 32, 8, 8192, 128, 512, "bf16", 1003, False, 1.0,
              1.0 / math.sqrt(128.0))
C3_WINDOWS = (128, 256, 512, 1024, 2048, 4096)
C4 = Workload("c4_train_step", 8, 16, 16, 4096, 128, 512, "bf16", 1004, True, 1.0,
              1.0 / math.sqrt(128.0))
C5 = Workload("c5_prefill_decode", 32, 32, 8, 32768, 128, 512, "bf16", 1005, False, 1.0,
              1.0 / math.sqrt(128.0), decode_steps=256)

WORKLOADS = {w.name: w for w in (C1, C2, C3, C4, C5)}


def _normal(shape, gen, device):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def _rows_to_unit_rms(x):
    return x / x.pow(2).mean(dim=-1, keepdim=True).sqrt()


def make_tensor(shape, seed, stream_id, dtype, device="cpu", unit_rms=False, mul=1.0):
    """One seeded N(0,1) tensor, drawn in fp32 one batch entry at a time (bounded scratch
    at the largest shapes), optionally row-normalised, then rounded to ``dtype``."""
    out = torch.empty(shape, dtype=dtype, device=device)
    for b in range(shape[0]):
        gen = torch.Generator(device=device)
        gen.manual_seed((seed * 1_000_003 + stream_id) * 4099 + b)
        x = _normal(shape[1:], gen, device)
        if unit_rms:
            x = _rows_to_unit_rms(x)
        if mul != 1.0:
            x = x * mul
        out[b] = x.to(dtype)
    return out


def make_qkv(wl: Workload, device="cpu"):
    """q [B,H_q,T,d], k, v [B,H_kv,T,d], already rounded to the workload's I/O type."""
    dt = wl.torch_dtype
    q = make_tensor((wl.B, wl.H_q, wl.T, wl.d), wl.seed, 0, dt, device, wl.qk_rms_norm,
                    wl.q_prescale)
    k = make_tensor((wl.B, wl.H_kv, wl.T, wl.d), wl.seed, 1, dt, device, wl.qk_rms_norm)
    v = make_tensor((wl.B, wl.H_kv, wl.T, wl.d), wl.seed, 2, dt, device)
    return q, k, v


def make_dout(wl: Workload, device="cpu"):
    """Upstream gradient dO ~ N(0,1), shape of the output."""
    return make_tensor((wl.B, wl.H_q, wl.T, wl.d), wl.seed, 3, wl.torch_dtype, device)


def make_decode_token(wl: Workload, step: int, device="cpu"):
    """Fresh q [B,H_q,d], k, v [B,H_kv,d] for decode step ``step``."""
    dt = wl.torch_dtype
    q = make_tensor((wl.B, wl.H_q, wl.d), wl.seed, 100 + 3 * step, dt, device,
                    wl.qk_rms_norm, wl.q_prescale)
    k = make_tensor((wl.B, wl.H_kv, wl.d), wl.seed, 101 + 3 * step, dt, device,
                    wl.qk_rms_norm)
    v = make_tensor((wl.B, wl.H_kv, wl.d), wl.seed, 102 + 3 * step, dt, device)
    return q, k, v


def make_gains(wl: Workload, device="cpu"):
    """Per-head RMS-norm gains [H_q, d] for both branches, near one (fp32)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(wl.seed * 7 + 5)
    gs = 1.0 + 0.1 * torch.randn((wl.H_q, wl.d), generator=gen)
    gr = 1.0 + 0.1 * torch.randn((wl.H_q, wl.d), generator=gen)
    return gs.to(device), gr.to(device)
