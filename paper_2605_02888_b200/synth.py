"""Seeded synthetic workloads shaped like the paper's speculation steps.

This module only makes INPUTS (logits, draft tokens, uniforms, per-row gamma / temperature,
controller weights).  It contains none of the method's arithmetic: no softmax, entropy,
acceptance test or inverse CDF.  Both the CUDA path and the test-side oracle read the bits
it produces (the oracle through a device-to-host copy), so neither side depends on how the
numbers were drawn.

Recipe (stands in for Llama-3.2 1B -> 3B logits, V = 128,256, gamma in {2,4,6,8}, three
compression levels, four task types; those models and prompts are not available here):
  target logit  t[v] = sigma_t * z[v] + 8 * rank(v)^-0.5 - s * ln rank(v),   z ~ N(0,1),
                rank(v) = 1 + ((a*v + c) mod V): an affine permutation of the vocabulary with a
                fixed multiplier a per task cluster and a fresh offset c per (step, row, position);
  draft logit   d[v] = t[v] + sigma_d * z'[v], rounded to the storage type after the add;
                sigma_d in {0.3, 0.6, 1.0} stands for an FP16 / INT8 / NF4 target (compression
                flags (0,0) / (1,0) / (0,1));
  draft token   x = argmax_v (d[v]/T + Gumbel noise)  (a draw from softmax(d/T)); plain argmax
                for greedy rows;
  uniforms      U[0,1) float32, two per position.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Optional, Sequence

import torch

SIGMA_LEVELS = (0.3, 0.6, 1.0)
GAMMA_CHOICES = (2, 4, 6, 8)


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    gamma_max: int
    V: int
    dtype: str = "bf16"                 # "bf16" | "fp32"
    steps: int = 1
    gamma_mode: str = "fixed"           # "fixed" | "choices" | "ragged" | "closed_loop"
    gamma_fixed: int = 4
    temperature: float = 1.0            # scalar temperature (ignored for temperature_mode "mixed")
    temperature_mode: str = "scalar"    # "scalar" | "mixed": 25% greedy rows, the rest U[0.6, 1.2]
    sigma_t: float = 2.0
    zipf_s: Sequence[float] = (1.1,)    # one exponent per task cluster; row b uses cluster (b % 12) // 3 if 4 given
    sigma_d: Sequence[float] = (0.5,)   # one value => every row; three => drawn per row
    frac_identical: float = 0.0         # rows whose draft equals the target bit for bit
    frac_onehot: float = 0.0            # rows with one token raised 30 above the row maximum
    seed: int = 0

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_bytes(self):
        return 2 if self.dtype == "bf16" else 4


# The five configurations of the benchmark definition (sizes, dtypes, distributions).
WORKLOADS = {
    "tiny": Workload("tiny", B=1, gamma_max=4, V=32000, dtype="fp32", steps=256, gamma_mode="fixed",
                     gamma_fixed=4, temperature=1.0, sigma_t=2.0, sigma_d=(0.5,)),
    "b64": Workload("b64", B=64, gamma_max=8, V=32000, dtype="bf16", steps=1000, gamma_mode="closed_loop",
                    gamma_fixed=4, temperature=1.0, sigma_t=2.0, sigma_d=SIGMA_LEVELS),
    "b256": Workload("b256", B=256, gamma_max=8, V=128256, dtype="bf16", steps=1, gamma_mode="choices",
                     temperature=0.8, sigma_t=2.5, sigma_d=SIGMA_LEVELS, frac_identical=0.10),
    # the same batch with every row at gamma = 8: the upper end of the headline configuration's traffic
    "b256_g8": Workload("b256_g8", B=256, gamma_max=8, V=128256, dtype="bf16", steps=1, gamma_mode="fixed",
                        gamma_fixed=8, temperature=0.8, sigma_t=2.5, sigma_d=SIGMA_LEVELS, frac_identical=0.10),
    "b512_mixed": Workload("b512_mixed", B=512, gamma_max=8, V=151936, dtype="fp32", steps=1,
                           gamma_mode="choices", temperature_mode="mixed", sigma_t=2.0, sigma_d=(0.5,),
                           frac_onehot=0.05),
    "b1024_loop": Workload("b1024_loop", B=1024, gamma_max=8, V=128256, dtype="bf16", steps=200,
                           gamma_mode="closed_loop", gamma_fixed=4, temperature=1.0, sigma_t=2.0,
                           zipf_s=(0.9, 1.1, 1.3, 1.6), sigma_d=SIGMA_LEVELS),
}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller or altered copy of a workload (tests use reduced B / V / steps)."""
    return replace(w, **kw)


@dataclass
class RowAttrs:
    """Per-row attributes that stay fixed over the steps of a run (CPU tensors)."""
    sigma_d: torch.Tensor      # [B] float32
    comp: torch.Tensor         # [B, 2] float32 compression flags
    cluster: torch.Tensor      # [B] int64 task cluster
    identical: torch.Tensor    # [B] bool
    onehot: torch.Tensor       # [B] bool
    onehot_token: torch.Tensor  # [B] int64
    temperature: torch.Tensor  # [B] float32 (0 => greedy)
    gamma0: torch.Tensor       # [B] int32 gamma of the first step


def row_attrs(w: Workload) -> RowAttrs:
    g = torch.Generator().manual_seed(w.seed * 7919 + 101)
    B = w.B
    n_cl = len(w.zipf_s)
    if n_cl == 4 and len(w.sigma_d) == 3:
        # 12 groups: group = b mod 12 -> (cluster, compression level)
        grp = torch.arange(B) % 12
        cluster = grp // 3
        level = grp % 3
    else:
        cluster = torch.arange(B) % n_cl
        level = torch.randint(0, len(w.sigma_d), (B,), generator=g)
    sig = torch.tensor(list(w.sigma_d), dtype=torch.float32)[level]
    comp = torch.zeros(B, 2)
    if len(w.sigma_d) == 3:
        comp[:, 0] = (level == 1).float()
        comp[:, 1] = (level == 2).float()
    r = torch.rand(B, 4, generator=g)
    identical = r[:, 0] < w.frac_identical
    onehot = r[:, 1] < w.frac_onehot
    onehot_token = torch.randint(0, w.V, (B,), generator=g)
    if w.temperature_mode == "mixed":
        T = 0.6 + 0.6 * r[:, 3]
        T = torch.where(r[:, 2] < 0.25, torch.zeros_like(T), T)
    else:
        T = torch.full((B,), float(w.temperature))
    if w.gamma_mode == "fixed" or w.gamma_mode == "closed_loop":
        gamma0 = torch.full((B,), min(w.gamma_fixed, w.gamma_max), dtype=torch.int32)
    elif w.gamma_mode == "choices":
        ch = torch.tensor([c for c in GAMMA_CHOICES if c <= w.gamma_max] or [w.gamma_max], dtype=torch.int32)
        gamma0 = ch[torch.randint(0, len(ch), (B,), generator=g)]
    elif w.gamma_mode == "ragged":
        gamma0 = torch.randint(1, w.gamma_max + 1, (B,), generator=g).to(torch.int32)
    else:
        raise ValueError(w.gamma_mode)
    return RowAttrs(sig, comp, cluster, identical, onehot, onehot_token, T.float(), gamma0)


_PRIMES = (1000003, 1000033, 1000037, 1000039)  # multipliers of the affine permutations (all > V)


def _rank_bias(w: Workload, device) -> torch.Tensor:
    """[n_cluster, V] float32: 8 * rank^-0.5 - s * ln(rank) laid out in permuted vocabulary order."""
    V = w.V
    rank = torch.arange(1, V + 1, dtype=torch.float64, device=device)
    v = torch.arange(V, dtype=torch.int64, device=device)
    out = []
    for k, s in enumerate(w.zipf_s):
        base = 8.0 * rank.pow(-0.5) - float(s) * rank.log()
        a = _PRIMES[k % len(_PRIMES)]
        while math.gcd(a, V) != 1:
            a += 2
        out.append(base[(a * v) % V].float())
    return torch.stack(out)


def make_mlp(w: Workload, device, n_in: int = 5, n_hidden: int = 16, n_out: int = 4):
    """Controller weights and biases ~ N(0, 0.1^2), one set per workload seed."""
    g = torch.Generator().manual_seed(w.seed * 7919 + 202)
    mk = lambda *s: (0.1 * torch.randn(*s, generator=g)).float().to(device)
    return dict(W1=mk(n_hidden, n_in), b1=mk(n_hidden), W2=mk(n_out, n_hidden), b2=mk(n_out))


def make_step(w: Workload, step: int, device, attrs: Optional[RowAttrs] = None,
              gamma: Optional[torch.Tensor] = None, rows_per_chunk: int = 64) -> dict:
    """Inputs of speculation step `step`: draft [B,G,V], target [B,G+1,V] (storage dtype),
    draft_tokens [B,G] int32, uniforms [B,G+1,2] fp32, gamma [B] int32, temperature [B] fp32,
    comp [B,2] fp32.  All gamma_max positions are generated whatever gamma is, so that two
    policies run on identical streams."""
    attrs = attrs or row_attrs(w)
    dev = torch.device(device)
    B, G, V = w.B, w.gamma_max, w.V
    dt = w.torch_dtype
    gen = torch.Generator(device=dev).manual_seed((w.seed * 1000003 + step) * 2 + 1)
    bias = _rank_bias(w, dev)                                   # [n_cluster, V]
    windows = torch.cat([bias, bias], dim=1).unfold(1, V, 1)    # [n_cluster, V+1, V] view: cyclic shifts
    target = torch.empty(B, G + 1, V, dtype=dt, device=dev)
    draft = torch.empty(B, G, V, dtype=dt, device=dev)
    tokens = torch.empty(B, G, dtype=torch.int32, device=dev)
    T = attrs.temperature.to(dev)
    sig = attrs.sigma_d.to(dev)
    cluster = attrs.cluster.to(dev)
    for r0 in range(0, B, rows_per_chunk):
        r1 = min(B, r0 + rows_per_chunk)
        n = r1 - r0
        shift = torch.randint(0, V, (n, G + 1), generator=gen, device=dev)
        t32 = w.sigma_t * torch.randn(n, G + 1, V, generator=gen, device=dev)
        t32 += windows[cluster[r0:r1, None].expand(n, G + 1), shift]
        hot = attrs.onehot[r0:r1].nonzero().flatten().tolist()
        for k in hot:
            tok = int(attrs.onehot_token[r0 + k])
            t32[k, :, tok] = t32[k].max(dim=-1).values + 30.0
        target[r0:r1] = t32.to(dt)
        d32 = t32[:, :G] + sig[r0:r1, None, None] * torch.randn(n, G, V, generator=gen, device=dev)
        d = d32.to(dt)
        same = attrs.identical[r0:r1].to(dev)
        d = torch.where(same[:, None, None], target[r0:r1, :G], d)
        draft[r0:r1] = d
        # draft tokens: Gumbel-max draw at the row temperature, argmax for greedy rows
        Tr = T[r0:r1, None, None]
        u = torch.rand(n, G, V, generator=gen, device=dev).clamp_(1e-20, 1.0 - 1e-7)
        gumbel = -(-(u.log())).log()
        z = d.float() / torch.where(Tr > 0, Tr, torch.ones_like(Tr)) + torch.where(Tr > 0, gumbel, torch.zeros_like(gumbel))
        tokens[r0:r1] = z.argmax(dim=-1).to(torch.int32)
        del t32, d32, d, u, gumbel, z
    uniforms = torch.rand(B, G + 1, 2, generator=gen, device=dev, dtype=torch.float32)
    gam = (attrs.gamma0 if gamma is None else gamma).to(device=dev, dtype=torch.int32)
    return dict(draft=draft, target=target, draft_tokens=tokens, uniforms=uniforms, gamma=gam,
                temperature=T.float().contiguous(), comp=attrs.comp.to(dev).contiguous())


def logit_bytes(w: Workload, gamma: torch.Tensor) -> int:
    """Algorithmic bytes of one step: every drafted position's draft row and every scored
    position's target row read once: sum_b (2*gamma_b + 1) * V * elem_bytes."""
    return int((2 * gamma.to(torch.int64) + 1).sum().item()) * w.V * w.elem_bytes
