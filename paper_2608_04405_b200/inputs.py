"""Seeded synthetic inputs for the BinaryPC decode path.

This module only produces *data*: key/value caches, queries, appended rows and
the Gaussian directions v* that Algorithm 1 draws.  It contains none of the
method's arithmetic (no hashing, scoring, selection or attention) and is the
only module that both the CUDA path's tests and the CPU checker read.

The paper evaluates on real model activations; those are not available, so the
workloads below stand in for them.  They take the shapes of the paper's models
(32/8 and 28/4 query/KV heads, head_dim 128, 32K-128K contexts, 2 % budget,
64/128-bit codes: Section 4 "Setup", Appendix "Hash bit length") and imitate
key statistics that matter for hashing: anisotropic channels, a few outlier
channels, a non-zero mean and rotary position encoding.

Recipe, per (sequence, KV head) unit:
  s_c  ~ LogNormal(0, 0.5)   channel scales, 4 distinct channels multiplied by 8
  mu_c ~ N(0, 0.5)           per-head mean (second parameter = std. deviation)
  K[i] = mu + s * z, z ~ N(0, I); V[i] ~ N(0, I)
  rotary encoding (rotate-half pairing c <-> c + D/2, theta_c = base^(-2c/D))
  applied to K at positions 0..n-1 when the workload has a rope base
  values rounded to the cache dtype (bf16 round-to-nearest-even, or fp32)
  query of a head = sum of m cached keys of its unit drawn without replacement
  + N(0, 0.1) noise, rounded to the cache dtype
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch

SEED_BASE = 2608044050  # per-workload seed = SEED_BASE + workload id


@dataclasses.dataclass(frozen=True)
class WorkloadSpec:
    name: str
    wid: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    n_ctx: int                  # context per sequence (upper bound when ragged)
    dtype: str                  # "bf16" | "f32"
    code_bits: int
    budget_ppm: int             # selected keys = ceil(n * ppm / 1e6)
    steps: int
    needles: int
    rope_base: Optional[float] = None
    n_ctx_min: Optional[int] = None   # ragged batches: lengths uniform in [n_ctx_min, n_ctx]
    head_dim: int = 128

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def esz(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    def scaled(self, **kw) -> "WorkloadSpec":
        return dataclasses.replace(self, **kw)


# The five synthetic configurations (shapes only; data comes from Workload).
CONFIGS = {
    0: WorkloadSpec("cfg0_tiny_fp32", 0, 1, 1, 1, 4096, "f32", 64, 20000, 16, 8),
    1: WorkloadSpec("cfg1_llama3_8b_32k", 1, 1, 32, 8, 32768, "bf16", 128, 20000, 256, 8, rope_base=500000.0),
    2: WorkloadSpec("cfg2_llama3_8b_128k_b4", 2, 4, 32, 8, 131072, "bf16", 128, 20000, 128, 16, rope_base=500000.0),
    3: WorkloadSpec("cfg3_ragged_b16", 3, 16, 32, 8, 65536, "bf16", 128, 20000, 64, 8, rope_base=500000.0,
                    n_ctx_min=16384),
    4: WorkloadSpec("cfg4_qwen25_7b_128k_b8", 4, 8, 28, 4, 131072, "bf16", 128, 20000, 512, 8, rope_base=1000000.0),
}


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def apply_rope(x: torch.Tensor, pos0: int, base: float) -> torch.Tensor:
    """Rotate-half rotary encoding of rows x[..., i, :] at positions pos0 + i (fp32 in, fp32 out)."""
    n, d = x.shape[-2], x.shape[-1]
    half = d // 2
    c = torch.arange(half, device=x.device, dtype=torch.float64)
    theta = base ** (-2.0 * c / d)
    pos = torch.arange(pos0, pos0 + n, device=x.device, dtype=torch.float64)
    ang = pos[:, None] * theta[None, :]
    cos, sin = torch.cos(ang).float(), torch.sin(ang).float()
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


class Workload:
    """Materialised caches and per-step inputs of one WorkloadSpec on one device.

    k_cache, v_cache : [batch, n_kv_heads, n_max, head_dim] in the cache dtype
    seq_lens         : python list of per-sequence context lengths (before any append)
    v_star           : [batch * n_kv_heads, code_bits, head_dim] fp32, the directions Algorithm 1 samples
    """

    def __init__(self, spec: WorkloadSpec, device="cpu", extra_rows: Optional[int] = None, salt: int = 0):
        self.spec = spec
        self.device = torch.device(device)
        s = spec
        seed = SEED_BASE + s.wid + 1000003 * salt
        self._seed = seed
        extra = s.steps + 64 if extra_rows is None else extra_rows
        self.n_max = ((s.n_ctx + extra + 63) // 64) * 64
        g = _gen(self.device, seed)
        U = s.batch * s.n_kv_heads
        D = s.head_dim
        if s.n_ctx_min is None:
            self.seq_lens: List[int] = [s.n_ctx] * s.batch
        else:
            lens = torch.randint(s.n_ctx_min, s.n_ctx + 1, (s.batch,), generator=_gen("cpu", seed + 17))
            self.seq_lens = [int(v) for v in lens]
        # per-unit channel statistics
        scale = torch.exp(0.5 * torch.randn(U, D, generator=g, device=self.device))
        for u in range(U):
            ch = torch.randperm(D, generator=g, device=self.device)[:4]
            scale[u, ch] *= 8.0
        self.scale = scale
        self.mean = 0.5 * torch.randn(U, D, generator=g, device=self.device)
        self.k_cache = torch.zeros(s.batch, s.n_kv_heads, self.n_max, D, dtype=s.torch_dtype, device=self.device)
        self.v_cache = torch.zeros_like(self.k_cache)
        for bi in range(s.batch):
            n = self.seq_lens[bi]
            for h in range(s.n_kv_heads):
                u = bi * s.n_kv_heads + h
                self.k_cache[bi, h, :n] = self._keys(u, 0, n, g)
                self.v_cache[bi, h, :n] = torch.randn(n, D, generator=g, device=self.device).to(s.torch_dtype)
        self.v_star = torch.randn(U, s.code_bits, D, generator=g, device=self.device)
        self._g = g

    def _keys(self, u: int, pos0: int, n: int, g: torch.Generator) -> torch.Tensor:
        s = self.spec
        z = torch.randn(n, s.head_dim, generator=g, device=self.device)
        k = self.mean[u] + self.scale[u] * z
        if s.rope_base is not None:
            k = apply_rope(k, pos0, s.rope_base)
        return k.to(s.torch_dtype)

    def new_kv(self, cur_lens: Sequence[int]):
        """One appended (k, v) row per unit, [batch, n_kv_heads, head_dim], at position cur_lens[b]."""
        s = self.spec
        k = torch.empty(s.batch, s.n_kv_heads, s.head_dim, dtype=s.torch_dtype, device=self.device)
        for bi in range(s.batch):
            for h in range(s.n_kv_heads):
                k[bi, h] = self._keys(bi * s.n_kv_heads + h, int(cur_lens[bi]), 1, self._g)[0]
        v = torch.randn(s.batch, s.n_kv_heads, s.head_dim, generator=self._g, device=self.device).to(s.torch_dtype)
        return k, v

    def queries(self, cur_lens: Sequence[int], k_cache: Optional[torch.Tensor] = None):
        """Queries [batch, n_q_heads, head_dim] planted on cached keys, plus the planted positions.

        Returns (q, needle_pos) with needle_pos [batch, n_q_heads, needles] (int64).
        """
        s = self.spec
        kc = self.k_cache if k_cache is None else k_cache
        q = torch.empty(s.batch, s.n_q_heads, s.head_dim, dtype=s.torch_dtype, device=self.device)
        pos = torch.empty(s.batch, s.n_q_heads, s.needles, dtype=torch.int64, device=self.device)
        for bi in range(s.batch):
            n = int(cur_lens[bi])
            for hq in range(s.n_q_heads):
                h = hq // s.group
                if n >= s.needles:
                    p = torch.randperm(n, generator=self._g, device=self.device)[: s.needles]
                else:                      # fewer cached keys than needles: draw with replacement
                    p = torch.randint(0, n, (s.needles,), generator=self._g, device=self.device)
                pos[bi, hq] = p
                vec = kc[bi, h, p].float().sum(0)
                vec = vec + 0.1 * torch.randn(s.head_dim, generator=self._g, device=self.device)
                q[bi, hq] = vec.to(s.torch_dtype)
        return q, pos


def algorithmic_bytes_per_step(spec: WorkloadSpec, seq_lens: Sequence[int]) -> int:
    """Bytes one decode step must move: packed codes of every cached key, the selected K and V rows, the queries
    and the outputs (Appendix "CUDA Optimizations": one code word per key; selected rows only).  The hash
    projection (b*D*esz per unit, about 1 % more) is read too but is not counted."""
    D, b, G = spec.head_dim, spec.code_bits, spec.group
    total = 0
    for n in seq_lens:
        k = min(n, -(-n * spec.budget_ppm // 1000000))
        per_unit = n * b // 8 + 2 * k * D * spec.esz + G * D * (spec.esz + 4)
        total += per_unit * spec.n_kv_heads
    return total
