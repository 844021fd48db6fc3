"""Seeded synthetic inputs shaped like the paper's workloads.

This module serves both the CUDA path and the CPU oracle's tests, so it holds none of the method's
arithmetic: only random draws, affine mixing of noise, and an arg-max.  Tokens "drawn from the
student softmax" use the Gumbel-max construction (arg-max of logits plus Gumbel noise), which needs
no softmax.

Recipes (standard deviations, not variances):
  config 1  B=2  T=64    V=4096    fp32  z~N(0,2)  u=z+N(0,1)            y~U[0,V)   W=[32,64]
  config 2  B=8  T=1024  V=32000   bf16  z~N(0,3)  u=0.8z+N(0,1.5)       y~p        W_b~U{128..1024}
  config 3  B=16 T=2048  V=151936  bf16  z~N(0,4)+10*Bern(0.05)  u=z+N(0,2)  y~p    W_b=256*2^(b%4)
  config 4  B=8  T=8192  V=151936  bf16  as config 3;  W_b~U{512..4096};  R_b=T or U{W_b..T}
  config 5  B=16 T=4096  V=151936  bf16  hidden states H_s [B,T,2048], H_t [B,T,2560] ~ N(0,1), output
            embeddings W_s [V,2048], W_t [V,2560] ~ N(0,0.02);  W_b~U{256..4096};  y~softmax(H_s W_s^T)
            (Gumbel-max over the products of the stored values, formed chunk by chunk with torch)
The teacher noise is added in fp32 to the unrounded student draw and both are then rounded to the
storage dtype.  Every sequence b has its own generator seeded with seed + 1000*config + b, so a
single sequence can be regenerated alone.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

SEED_BASE = 20260528

CONFIGS = {
    1: dict(B=2, T=64, V=4096, dtype="f32", s_std=2.0, mix=1.0, t_std=1.0, spike_p=0.0,
            tokens="uniform"),
    2: dict(B=8, T=1024, V=32000, dtype="bf16", s_std=3.0, mix=0.8, t_std=1.5, spike_p=0.0,
            tokens="student"),
    3: dict(B=16, T=2048, V=151936, dtype="bf16", s_std=4.0, mix=1.0, t_std=2.0, spike_p=0.05,
            tokens="student"),
    4: dict(B=8, T=8192, V=151936, dtype="bf16", s_std=4.0, mix=1.0, t_std=2.0, spike_p=0.05,
            tokens="student"),
}
SPIKE = 10.0


@dataclass
class Batch:
    student: torch.Tensor      # [B,T,V]
    teacher: torch.Tensor      # [B,T,V]
    tokens: torch.Tensor       # [B,T] int32
    window: torch.Tensor       # [B] int32
    rollout_len: torch.Tensor  # [B] int32
    config: int

    @property
    def shape(self):
        return tuple(self.student.shape)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def windows_for(config: int, B: int, T: int, seed: int = SEED_BASE, ragged_rollout: bool = False):
    """Window and rollout lengths of a config (host int32 tensors)."""
    g = _gen("cpu", seed + 1000 * config + 999)
    if config == 1:
        w = torch.tensor([T // 2, T][:B] + [T] * max(0, B - 2), dtype=torch.int32)
    elif config == 2:
        lo = min(128, T)
        w = torch.randint(lo, T + 1, (B,), generator=g, dtype=torch.int32)
    elif config == 3:
        tiers = [T // 8, T // 4, T // 2, T]
        w = torch.tensor([max(1, tiers[b % 4]) for b in range(B)], dtype=torch.int32)
    elif config == 4:
        lo, hi = max(1, T // 16), max(1, T // 2)
        w = torch.randint(lo, hi + 1, (B,), generator=g, dtype=torch.int32)
    else:
        raise ValueError(config)
    if ragged_rollout:
        r = torch.stack([torch.randint(int(wb), T + 1, (1,), generator=g, dtype=torch.int32)[0]
                         for wb in w])
    else:
        r = torch.full((B,), T, dtype=torch.int32)
    return w, r.to(torch.int32)


def fill_sequence(student_b, teacher_b, tokens_b, *, s_std, mix, t_std, spike_p, tokens, gen,
                  rows_per_chunk=256):
    """Fill one sequence's [T,V] logits and [T] tokens in place, chunked over rows."""
    T, V = student_b.shape
    dev = student_b.device
    for t0 in range(0, T, rows_per_chunk):
        t1 = min(T, t0 + rows_per_chunk)
        n = t1 - t0
        z = torch.randn((n, V), generator=gen, device=dev, dtype=torch.float32) * s_std
        if spike_p > 0:
            z += SPIKE * (torch.rand((n, V), generator=gen, device=dev) < spike_p)
        u = mix * z + t_std * torch.randn((n, V), generator=gen, device=dev, dtype=torch.float32)
        student_b[t0:t1] = z.to(student_b.dtype)
        teacher_b[t0:t1] = u.to(teacher_b.dtype)
        if tokens == "uniform":
            tokens_b[t0:t1] = torch.randint(0, V, (n,), generator=gen, device=dev,
                                            dtype=torch.int32)
        else:
            e = torch.rand((n, V), generator=gen, device=dev, dtype=torch.float32)
            e = e.clamp_(min=1e-20).log_().neg_().log_().neg_()        # Gumbel(0,1)
            e += student_b[t0:t1].to(torch.float32)                    # stored (rounded) logits
            tokens_b[t0:t1] = e.argmax(dim=1).to(torch.int32)
        del z, u


def make_batch(config: int, device="cpu", seed: int = SEED_BASE, B=None, T=None, V=None,
               ragged_rollout: bool = False, fill_all_rows: bool = True) -> Batch:
    """Inputs of one config, optionally at reduced B/T/V (same recipe, smaller shape).

    With fill_all_rows=False only rows t < R_b are generated (the rest stay zero); rows past the
    rollout are never read by the method, so this only saves generation time.
    """
    spec = dict(CONFIGS[config])
    B = spec["B"] if B is None else B
    T = spec["T"] if T is None else T
    V = spec["V"] if V is None else V
    dt = torch.float32 if spec["dtype"] == "f32" else torch.bfloat16
    student = torch.zeros((B, T, V), dtype=dt, device=device)
    teacher = torch.zeros((B, T, V), dtype=dt, device=device)
    tokens = torch.zeros((B, T), dtype=torch.int32, device=device)
    window, rollout = windows_for(config, B, T, seed, ragged_rollout)
    for b in range(B):
        gen = _gen(device, seed + 1000 * config + b)
        n = T if fill_all_rows else int(rollout[b])
        if n > 0:
            fill_sequence(student[b, :n], teacher[b, :n], tokens[b, :n], s_std=spec["s_std"],
                          mix=spec["mix"], t_std=spec["t_std"], spike_p=spec["spike_p"],
                          tokens=spec["tokens"], gen=gen)
    return Batch(student, teacher, tokens, window.to(device), rollout.to(device), config)


def bits_for_oracle(x: torch.Tensor):
    """Stored logits as the numpy array the oracle accepts (float32, or uint16 bf16 bits)."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.float32:
        return x.numpy()
    if x.dtype == torch.bfloat16:
        import numpy as np
        return x.view(torch.int16).numpy().view(np.uint16)
    raise TypeError(x.dtype)


LMHEAD = dict(B=16, T=4096, V=151936, d_s=2048, d_t=2560, h_std=1.0, w_std=0.02)


@dataclass
class LmHeadBatch:
    hidden_student: torch.Tensor   # [B,T,d_s] bf16
    w_student: torch.Tensor        # [V,d_s]   bf16
    hidden_teacher: torch.Tensor   # [B,T,d_t] bf16
    w_teacher: torch.Tensor        # [V,d_t]   bf16
    tokens: torch.Tensor           # [B,T] int32
    window: torch.Tensor           # [B] int32
    rollout_len: torch.Tensor      # [B] int32


def make_lmhead_batch(device="cpu", seed: int = SEED_BASE, B=None, T=None, V=None, d_s=None,
                      d_t=None, w_std=None, ragged_rollout: bool = False,
                      rows_per_chunk: int = 512) -> LmHeadBatch:
    """Inputs of config 5 (fused LM-head variant), optionally at reduced shape.

    Tokens are drawn from the student softmax with the Gumbel-max construction; the products
    H_s W_s^T needed for that are taken in fp32 over the stored bf16 values, a block of rows at a
    time, and only for positions inside the rollout (the rest keep token 0).
    """
    spec = LMHEAD
    B = spec["B"] if B is None else B
    T = spec["T"] if T is None else T
    V = spec["V"] if V is None else V
    d_s = spec["d_s"] if d_s is None else d_s
    d_t = spec["d_t"] if d_t is None else d_t
    w_std = spec["w_std"] if w_std is None else w_std
    g = _gen(device, seed + 5000 + 4242)      # apart from the per-sequence seeds below
    ws = (torch.randn((V, d_s), generator=g, device=device, dtype=torch.float32) * w_std)
    ws = ws.to(torch.bfloat16)
    wt = (torch.randn((V, d_t), generator=g, device=device, dtype=torch.float32) * w_std)
    wt = wt.to(torch.bfloat16)
    gw = _gen("cpu", seed + 5000 + 999)
    lo = max(1, T // 16)
    window = torch.randint(lo, T + 1, (B,), generator=gw, dtype=torch.int32)
    if ragged_rollout:
        rollout = torch.stack([torch.randint(int(wb), T + 1, (1,), generator=gw,
                                             dtype=torch.int32)[0] for wb in window])
    else:
        rollout = torch.full((B,), T, dtype=torch.int32)
    hs = torch.empty((B, T, d_s), dtype=torch.bfloat16, device=device)
    ht = torch.empty((B, T, d_t), dtype=torch.bfloat16, device=device)
    tokens = torch.zeros((B, T), dtype=torch.int32, device=device)
    ws32 = ws.to(torch.float32) if V * d_s <= (1 << 26) else None
    for b in range(B):
        gb = _gen(device, seed + 5000 + b)
        hs[b] = (torch.randn((T, d_s), generator=gb, device=device, dtype=torch.float32)
                 * spec["h_std"]).to(torch.bfloat16)
        ht[b] = (torch.randn((T, d_t), generator=gb, device=device, dtype=torch.float32)
                 * spec["h_std"]).to(torch.bfloat16)
        n = int(rollout[b])
        for t0 in range(0, n, rows_per_chunk):
            t1 = min(n, t0 + rows_per_chunk)
            h = hs[b, t0:t1]
            if ws32 is not None:
                z = h.to(torch.float32) @ ws32.T
            else:
                z = (h @ ws.T).to(torch.float32)
            e = torch.rand(z.shape, generator=gb, device=device, dtype=torch.float32)
            e = e.clamp_(min=1e-20).log_().neg_().log_().neg_()
            z += e
            tokens[b, t0:t1] = z.argmax(dim=1).to(torch.int32)
            del z, e
    return LmHeadBatch(hs, ws, ht, wt, tokens, window.to(device), rollout.to(torch.int32).to(device))
