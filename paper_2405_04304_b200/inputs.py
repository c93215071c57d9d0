"""Seeded synthetic inputs for the DISCO logit tails.

This module only draws random numbers and packs them.  It contains none of the
method's arithmetic (no projection, soft-max, classifier or prefix match), so
it can feed the CUDA library, a CPU checker and the benchmark alike without
making any of them depend on another.  It never loads the CUDA library.

The workloads mirror the model pairs the paper evaluates (Vicuna-13B/68M and
Starcoder-15B/168M, Sec. 4): only the shapes of their LM heads and hidden
states matter here, weights and activations are Gaussian.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

N_FEAT = 12  # Eq. 2: top-10 probabilities, entropy, position


@dataclass(frozen=True)
class Workload:
    name: str
    V: int            # vocabulary size
    d_D: int          # draft hidden width
    d_T: int          # target hidden width
    B: int            # independent sequences
    sl_max: int       # cap on drafted tokens per iteration
    iterations: int
    p_corrupt: float  # per-position probability that a draft id is replaced by a random id
    tau: float = 0.5
    H: int = 64       # classifier hidden width
    seed: int = 0
    sl_mode: str = "classifier"   # "classifier": SL decided by the halt flag; "uniform": forced SL_b ~ U{1..sl_max}
    accept_beta: tuple | None = None  # (a, b): per-sequence acceptance rate ~ Beta(a, b), overrides p_corrupt

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    "tiny": Workload("tiny", V=32000, d_D=768, d_T=2048, B=1, sl_max=5, iterations=16,
                     p_corrupt=0.2, seed=0),
    "vicuna_b1": Workload("vicuna_b1", V=32000, d_D=768, d_T=5120, B=1, sl_max=10,
                          iterations=256, p_corrupt=0.2, seed=1),
    "starcoder_b1": Workload("starcoder_b1", V=49152, d_D=768, d_T=6144, B=1, sl_max=10,
                             iterations=256, p_corrupt=0.1, seed=2),
    "vicuna_b64": Workload("vicuna_b64", V=32000, d_D=768, d_T=5120, B=64, sl_max=10,
                           iterations=64, p_corrupt=0.3, seed=3, sl_mode="uniform"),
    "starcoder_b256": Workload("starcoder_b256", V=49152, d_D=768, d_T=6144, B=256, sl_max=16,
                               iterations=64, p_corrupt=0.0, seed=4, accept_beta=(4.0, 2.0)),
}


def _gen(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def sub_seed(seed: int, *tags: int) -> int:
    """Deterministic child seed for (seed, tags...); plain integer mixing."""
    s = (int(seed) + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
    for t in tags:
        s ^= (int(t) + 0x9E3779B97F4A7C15 + ((s << 6) & 0xFFFFFFFFFFFFFFFF) + (s >> 2)) & 0xFFFFFFFFFFFFFFFF
        s = (s * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        s ^= s >> 31
    return s & 0x7FFFFFFFFFFFFFFF


def lm_head(V: int, d: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    """bf16 [V, d] ~ N(0, std^2).  Drawn in chunks so that no fp32 copy of a large head is held."""
    out = torch.empty((V, d), dtype=torch.bfloat16, device=device)
    g = _gen(seed, device)
    rows = max(1, (1 << 24) // max(d, 1))
    for v0 in range(0, V, rows):
        v1 = min(V, v0 + rows)
        out[v0:v1] = (torch.randn((v1 - v0, d), generator=g, device=device, dtype=torch.float32)
                      * std).to(torch.bfloat16)
    return out


def hidden(R: int, d: int, seed: int, device="cpu") -> torch.Tensor:
    """bf16 [R, d] ~ N(0, 1)."""
    g = _gen(seed, device)
    return torch.randn((R, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def classifier_params(H: int, seed: int, n_feat: int = N_FEAT):
    """fp32 (W1 [H,n_feat], b1 [H], w2 [H], b2 [1]), each U(-1/sqrt(fan_in), +1/sqrt(fan_in))."""
    g = _gen(seed)

    def u(shape, fan_in):
        bound = 1.0 / float(np.sqrt(fan_in))
        return (torch.rand(shape, generator=g, dtype=torch.float32) * 2.0 - 1.0) * bound

    return u((H, n_feat), n_feat), u((H,), n_feat), u((H,), H), u((1,), H)


def corrupt_ids(ids: torch.Tensor, p, V: int, seed: int) -> torch.Tensor:
    """Replace each id, independently with probability p, by a uniform id in [0, V).

    ``p`` is a float or a tensor broadcastable to ``ids`` (per-position probabilities)."""
    g = _gen(seed)
    ids = ids.to("cpu", torch.int32)
    coin = torch.rand(ids.shape, generator=g)
    rnd = torch.randint(0, V, ids.shape, generator=g, dtype=torch.int32)
    p = torch.as_tensor(p, dtype=torch.float32)
    return torch.where(coin < p, rnd, ids)


def uniform_sl(B: int, lo: int, hi: int, seed: int) -> torch.Tensor:
    """int32 [B], each uniform in {lo..hi}."""
    return torch.randint(lo, hi + 1, (B,), generator=_gen(seed), dtype=torch.int32)


def beta_rates(B: int, a: float, b: float, seed: int) -> torch.Tensor:
    """float32 [B] ~ Beta(a, b) from two Gamma draws."""
    rng = np.random.Generator(np.random.PCG64(int(seed)))
    return torch.from_numpy(rng.beta(a, b, size=B).astype(np.float32))


def row_offsets(sl: torch.Tensor) -> torch.Tensor:
    """int32 [B+1]: exclusive prefix sum of (SL_b + 1)."""
    off = torch.zeros(sl.numel() + 1, dtype=torch.int32)
    off[1:] = torch.cumsum(sl.to(torch.int32) + 1, 0)
    return off


def pack_rows(H_full: torch.Tensor, sl: torch.Tensor, sl_max: int) -> torch.Tensor:
    """Keep the first SL_b+1 of each sequence's sl_max+1 rows; [B*(sl_max+1), d] -> [R, d]."""
    B = sl.numel()
    d = H_full.shape[1]
    H3 = H_full.view(B, sl_max + 1, d)
    return torch.cat([H3[b, : int(sl[b]) + 1] for b in range(B)], 0).contiguous()


def pack_ids(ids_full: torch.Tensor, sl: torch.Tensor, sl_max: int) -> torch.Tensor:
    """Keep the first SL_b of each sequence's sl_max draft ids; [B*sl_max] -> [R-B]."""
    B = sl.numel()
    I2 = ids_full.view(B, sl_max)
    parts = [I2[b, : int(sl[b])] for b in range(B)]
    return torch.cat(parts, 0).contiguous() if parts else ids_full[:0]


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)
