"""Seeded synthetic inputs shaped like the paper's long-context workloads.

This module only makes inputs (random bf16 Q/K/V, planted heavy keys, head
masks, decode-step tensors).  It holds none of the method's arithmetic and is
the one module that both the CPU oracle's tests and the CUDA path's tests and
benchmark import.  Every tensor is a function of (workload seed, layer, step,
tensor name) only; a tensor is generated once, on one device, and the same
bits are handed to both sides.

The paper evaluates on RULER, LongBench and Needle-in-a-Haystack with trained
models; none of that is available here, so these inputs stand in for them and
only the shapes are taken from the paper's setting (Llama-3-8B / Qwen2.5-7B
attention shapes, 32K-256K contexts, budgets 1024-4096, observation windows
32/64).
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np
import torch

POOL_NONE, POOL_CHUNK, POOL_SLIDING = 0, 1, 2
N_HEAVY = 16


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    B: int
    Hq: int
    Hkv: int
    n: int                     # prefill context length
    L_obs: int                 # observation window
    consistent_lo: float       # share of consistent KV heads (per sequence: drawn in [lo, hi])
    consistent_hi: float
    budget: int                # token budget of a consistent head
    eta: float                 # retention ratio of an adaptive head (1.0 = full cache)
    pool_mode: int
    pool_param: int
    decode_steps: int
    seed: int
    d: int = 128
    sink: int = 4
    local: int = 64

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


WORKLOADS: Dict[str, Workload] = {
    # configs[0]: single layer, 4 of 8 KV heads consistent at budget 256 = sink 4 + local 64 + 188 top-k
    "cfg0": Workload("cfg0", 1, 1, 32, 8, 4096, 32, 0.5, 0.5, 256, 1.0, POOL_NONE, 0, 16, 1000),
    # configs[1]: Llama-3-8B shape, 32K context, 50 % consistent at 1024, sliding max-pool 7
    "cfg1": Workload("cfg1", 32, 1, 32, 8, 32768, 32, 0.5, 0.5, 1024, 1.0, POOL_SLIDING, 7, 128, 1001),
    # configs[2]: 128K context, 60 % consistent at 2048, adaptive heads keep 90 %
    "cfg2": Workload("cfg2", 32, 1, 32, 8, 131072, 32, 0.6, 0.6, 2048, 0.9, POOL_SLIDING, 7, 128, 1002),
    # configs[3]: batch 16 x 64K, per-sequence masks with 40-70 % consistent heads, budget 1024
    "cfg3": Workload("cfg3", 32, 16, 32, 8, 65536, 32, 0.4, 0.7, 1024, 1.0, POOL_SLIDING, 7, 64, 1003),
    # configs[4]: Qwen2.5-7B shape, batch 4 x 256K, GQA 7, 50 % consistent at 4096, window 64, chunks of 8
    "cfg4": Workload("cfg4", 28, 4, 28, 4, 262144, 64, 0.5, 0.5, 4096, 1.0, POOL_CHUNK, 8, 16, 1004),
}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller (or otherwise altered) copy of a workload, for tests."""
    return replace(w, **kw)


def _seed(*parts) -> int:
    h = hashlib.sha256(("|".join(str(p) for p in parts)).encode()).digest()
    return int.from_bytes(h[:8], "little") & 0x7FFFFFFFFFFFFFFF


def _gen(device, *parts) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*parts))
    return g


def _rng(*parts) -> np.random.Generator:
    return np.random.default_rng(_seed(*parts))


def randn_bf16(shape, device, *parts) -> torch.Tensor:
    """N(0,1) values rounded once to bf16."""
    g = _gen(device, *parts)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def head_mask(w: Workload, layer: int) -> np.ndarray:
    """[B, Hkv] uint8, 1 = consistent.  The share of consistent heads of a
    sequence is drawn in [consistent_lo, consistent_hi]; share * Hkv is rounded
    stochastically to a head count (so the share holds on average over
    layers); which heads is a seeded permutation."""
    rng = _rng(w.seed, "mask", layer)
    m = np.zeros((w.B, w.Hkv), dtype=np.uint8)
    for b in range(w.B):
        frac = w.consistent_lo + (w.consistent_hi - w.consistent_lo) * rng.random()
        x = frac * w.Hkv
        cnt = int(math.floor(x)) + (1 if rng.random() < x - math.floor(x) else 0)
        m[b, rng.permutation(w.Hkv)[:cnt]] = 1
    return m


def directions(w: Workload, layer: int, device) -> torch.Tensor:
    """One unit direction per (sequence, KV head): [B, Hkv, d] float32."""
    c = torch.randn((w.B, w.Hkv, w.d), generator=_gen(device, w.seed, "dir", layer), device=device)
    return c / c.norm(dim=-1, keepdim=True)


def heavy_positions(w: Workload, layer: int, n: Optional[int] = None) -> np.ndarray:
    """[B, Hkv, 16] distinct token positions inside the candidate range [sink, n - local)."""
    n = w.n if n is None else n
    rng = _rng(w.seed, "heavy", layer)
    lo, hi = w.sink, n - max(w.local, w.L_obs)
    pos = np.zeros((w.B, w.Hkv, N_HEAVY), dtype=np.int64)
    for b in range(w.B):
        for h in range(w.Hkv):
            pos[b, h] = np.sort(rng.choice(hi - lo, size=min(N_HEAVY, hi - lo), replace=False) + lo)
    return pos


def boost(w: Workload) -> float:
    """s = t with s*t = 4*sqrt(d): adding s*c to a key and t*c to a query lifts
    their scaled logit by +4, four standard deviations of an N(0,1) logit."""
    return math.sqrt(4.0 * math.sqrt(w.d))


def prefill_layer(w: Workload, layer: int, device="cpu", with_v: bool = True):
    """Prefill tensors of one layer.

    Returns dict: q_win [B, Hq, L_obs, d], k, v [B, Hkv, n, d] (bf16),
    seq_len [B] (all n), head_mask [B, Hkv], heavy [B, Hkv, 16].
    Keys at the heavy positions get +s*c_h, the window queries of the group
    get +t*c_h.
    """
    s = boost(w)
    c = directions(w, layer, device)
    pos = heavy_positions(w, layer)
    k = torch.empty((w.B, w.Hkv, w.n, w.d), dtype=torch.bfloat16, device=device)
    v = torch.empty((w.B, w.Hkv, w.n, w.d), dtype=torch.bfloat16, device=device) if with_v else None
    for b in range(w.B):  # per sequence: bounds the fp32 temporaries
        k[b] = randn_bf16((w.Hkv, w.n, w.d), device, w.seed, "k", layer, b)
        if with_v:
            v[b] = randn_bf16((w.Hkv, w.n, w.d), device, w.seed, "v", layer, b)
    pos_t = torch.from_numpy(pos).to(device)
    for b in range(w.B):
        for h in range(w.Hkv):
            rows = k[b, h, pos_t[b, h]].float() + s * c[b, h][None, :]
            k[b, h, pos_t[b, h]] = rows.to(torch.bfloat16)
    q = torch.randn((w.B, w.Hq, w.L_obs, w.d), generator=_gen(device, w.seed, "qwin", layer), device=device)
    q = q + s * c.repeat_interleave(w.G, dim=1)[:, :, None, :]
    return {
        "q_win": q.to(torch.bfloat16), "k": k, "v": v,
        "seq_len": np.full((w.B,), w.n, dtype=np.int32),
        "head_mask": head_mask(w, layer), "heavy": pos,
    }


def decode_inputs(w: Workload, layer: int, step: int, device="cpu", mask: Optional[np.ndarray] = None):
    """q [B, Hq, d], k_new, v_new [B, Hkv, d] (bf16) of one decode step.  The
    decode queries of consistent heads lean on the head's direction, as the
    window queries did (sequential consistency)."""
    q = torch.randn((w.B, w.Hq, w.d), generator=_gen(device, w.seed, "q", layer, step), device=device)
    mask = head_mask(w, layer) if mask is None else mask
    c = directions(w, layer, device)
    lean = torch.from_numpy(mask.astype(np.float32)).to(device)[:, :, None] * c * boost(w)
    q = q + lean.repeat_interleave(w.G, dim=1)
    kn = randn_bf16((w.B, w.Hkv, w.d), device, w.seed, "kn", layer, step)
    vn = randn_bf16((w.B, w.Hkv, w.d), device, w.seed, "vn", layer, step)
    return q.to(torch.bfloat16), kn, vn


def calibration_prompt(w: Workload, layer: int, prompt: int, n: int, types: np.ndarray, device="cpu",
                       n_heavy_rows: int = 4):
    """One calibration prompt for head identification: q_win [1, Hq, L_obs, d],
    k [1, Hkv, n, d].

    types [Hkv] (1 = consistent).  A consistent head shares one direction and
    one set of 16 heavy keys across all window rows (similar rows, few
    columns); an adaptive head gives every window row its own direction and
    its own heavy keys, so no column is hit by many rows.
    """
    s = boost(w)
    rng = _rng(w.seed, "calib", layer, prompt)
    k = randn_bf16((1, w.Hkv, n, w.d), device, w.seed, "ck", layer, prompt)
    q = torch.randn((1, w.Hq, w.L_obs, w.d), generator=_gen(device, w.seed, "cq", layer, prompt), device=device)
    lo, hi = n // 32, n - 2 * w.L_obs
    for h in range(w.Hkv):
        if types[h]:
            c = torch.randn((w.d,), generator=_gen(device, w.seed, "cd", layer, prompt, h), device=device)
            c = c / c.norm()
            pos = torch.from_numpy(np.sort(rng.choice(hi - lo, N_HEAVY, replace=False) + lo)).to(device)
            k[0, h, pos] = (k[0, h, pos].float() + s * c[None, :]).to(torch.bfloat16)
            q[0, h * w.G:(h + 1) * w.G] += s * c[None, None, :]
        else:
            c = torch.randn((w.L_obs, w.d), generator=_gen(device, w.seed, "cd", layer, prompt, h), device=device)
            c = c / c.norm(dim=-1, keepdim=True)
            for i in range(w.L_obs):
                pos = torch.from_numpy(np.sort(rng.choice(hi - lo, n_heavy_rows, replace=False) + lo)).to(device)
                k[0, h, pos] = (k[0, h, pos].float() + s * c[i][None, :]).to(torch.bfloat16)
            q[0, h * w.G:(h + 1) * w.G] += s * c[None, :, :]
    return q.to(torch.bfloat16), k


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host copy)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)
