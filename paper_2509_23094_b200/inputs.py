"""Seeded synthetic inputs for the d2Cache decode step.

This module only *draws* inputs (shapes, random weights, token ids, mask
patterns, score vectors).  It holds none of the method's arithmetic: no
density, no selection, no transformer math.  Both the CPU oracle's tests and
the CUDA path's tests feed from it so that the two sides see identical bytes.

The workloads are synthetic stand-ins for the paper's evaluation prompts run
through trained LLaDA-8B / Dream-7B checkpoints (Section 5.1): random weights
of the named shapes, uniform random token ids, and mask patterns with the
structure the paper's decoding produces (a known prompt followed by a
generation region that is partly decoded, partly still masked).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional

import torch


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float
    rms_eps: float
    qkv_bias: bool

    @property
    def qkv_out(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def params_per_layer(self) -> int:
        d, hd = self.d_model, self.head_dim
        return d * self.qkv_out + self.n_q_heads * hd * d + 3 * d * self.d_ffn


TOY = ModelShape("toy", 1, 256, 4, 4, 64, 768, 1024, 10000.0, 1e-5, False)
# Same family as TOY but several layers, grouped KV heads and a QKV bias: small
# enough for the oracle, exercises every code path the large shapes do.
TOY_GQA = ModelShape("toy_gqa", 3, 256, 4, 2, 64, 512, 640, 10000.0, 1e-6, True)
TOY_HD128 = ModelShape("toy_hd128", 2, 512, 4, 2, 128, 1024, 1000, 10000.0, 1e-5, False)
LLADA_8B_1L = ModelShape("llada8b_1layer", 1, 4096, 32, 32, 128, 12288, 126464, 500000.0, 1e-5, False)
LLADA_8B = replace(LLADA_8B_1L, name="llada8b", n_layers=32)
DREAM_7B = ModelShape("dream7b", 28, 3584, 28, 4, 128, 18944, 152064, 1.0e6, 1e-6, True)


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    batch: int
    seq_len: int
    prompt_len: int
    n_masked: int          # per sequence, inside the generation region
    mask_pattern: str      # "random" | "suffix" (semi-AR: trailing slots masked) | "all"
    k: int
    p: float
    seed: int = 0
    sigma: float = 10.0


WORKLOADS: Dict[str, Workload] = {
    # config 1: toy single layer, 64 prompt + 64 slots, 32 of them masked at random
    "toy": Workload("toy", TOY, 1, 128, 64, 32, "random", 8, 0.9),
    # config 2: one LLaDA-8B-shaped layer, 768 prompt + 256 slots decoded
    # left to right in blocks of 32, the last 128 slots still masked
    "llada1l_1024": Workload("llada1l_1024", LLADA_8B_1L, 1, 1024, 768, 128, "suffix", 32, 0.9),
    # config 3: full LLaDA-8B shape, 512 prompt + 256 masked slots, decode loop
    "llada_decode": Workload("llada_decode", LLADA_8B, 1, 768, 512, 256, "all", 32, 0.9),
    # config 4: Dream-7B shape, batch 4, 1024 prompt + 512 masked slots
    "dream_decode": Workload("dream_decode", DREAM_7B, 4, 1536, 1024, 512, "all", 64, 0.9),
    # config 5: long-context stress, batch 8 x 4096, half of 1024 slots masked
    "llada_long": Workload("llada_long", LLADA_8B, 8, 4096, 3072, 512, "random", 64, 0.8),
}


def _gen(seed: int, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal_bf16(shape, std: float, g: torch.Generator, device: str) -> torch.Tensor:
    """bf16(N(0, std^2)), drawn in chunks so huge tensors never need an fp32 copy."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    chunk = 1 << 26
    for s in range(0, flat.numel(), chunk):
        e = min(s + chunk, flat.numel())
        flat[s:e] = (torch.randn(e - s, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out


def make_weights(shape: ModelShape, seed: int = 0, device: str = "cpu", std: float = 0.02,
                 gain_jitter: float = 0.0, with_embed: bool = True,
                 share_layers: bool = False) -> Dict[str, object]:
    """Random-init weights of the given shape, all bf16, matrices stored [out][in].

    gain_jitter > 0 draws RMSNorm gains as 1 + jitter*N(0,1) (tests use this so
    a dropped gain shows up); the workloads keep gains at 1.
    share_layers=True draws one layer and aliases it n_layers times (used only
    where a full-depth model would not fit next to its own copy).
    """
    g = _gen(seed, device)
    d, F = shape.d_model, shape.d_ffn

    def gain():
        if gain_jitter > 0:
            return (1.0 + gain_jitter * torch.randn(d, generator=g, device=device)).to(torch.bfloat16)
        return torch.ones(d, dtype=torch.bfloat16, device=device)

    def layer():
        return {
            "g_attn": gain(),
            "wqkv": _normal_bf16((shape.qkv_out, d), std, g, device),
            "bqkv": _normal_bf16((shape.qkv_out,), std, g, device) if shape.qkv_bias else None,
            "wo": _normal_bf16((d, shape.n_q_heads * shape.head_dim), std, g, device),
            "g_ffn": gain(),
            "w_gate": _normal_bf16((F, d), std, g, device),
            "w_up": _normal_bf16((F, d), std, g, device),
            "w_down": _normal_bf16((d, F), std, g, device),
        }

    if share_layers:
        one = layer()
        layers: List[dict] = [one for _ in range(shape.n_layers)]
    else:
        layers = [layer() for _ in range(shape.n_layers)]
    w: Dict[str, object] = {"layers": layers, "g_final": gain(),
                            "w_lm": _normal_bf16((shape.vocab, d), std, g, device)}
    if with_embed:
        w["embed"] = _normal_bf16((shape.vocab, d), std, g, device)
    return w


def make_mask(wl: Workload, device: str = "cpu") -> torch.Tensor:
    """uint8 [batch][seq_len], 1 = still [MASK]; pattern drawn per sequence from seed+b."""
    B, L, P = wl.batch, wl.seq_len, wl.prompt_len
    slots = L - P
    mask = torch.zeros(B, L, dtype=torch.uint8)
    for b in range(B):
        if wl.mask_pattern == "all":
            mask[b, P:] = 1
        elif wl.mask_pattern == "suffix":
            mask[b, L - wl.n_masked:] = 1
        elif wl.mask_pattern == "random":
            perm = torch.randperm(slots, generator=_gen(wl.seed + 1000 + b))
            mask[b, P + perm[: wl.n_masked]] = 1
        else:
            raise ValueError(wl.mask_pattern)
    return mask.to(device)


def make_tokens(wl: Workload, mask: torch.Tensor) -> torch.Tensor:
    """int64 [batch][seq_len]: uniform ids over [0, vocab-1); masked slots hold the reserved id vocab-1."""
    g = _gen(wl.seed + 2000)
    tok = torch.randint(0, wl.shape.vocab - 1, (wl.batch, wl.seq_len), generator=g)
    tok[mask.cpu().bool()] = wl.shape.vocab - 1
    return tok


def make_h0(embed: torch.Tensor, tokens: torch.Tensor) -> torch.Tensor:
    """bf16 [batch][seq_len][d]: embedding rows of the tokens (a table lookup, no arithmetic)."""
    return embed[tokens.to(embed.device)].contiguous()


def make_scores(n: int, seed: int, kind: str = "uniform", ties: int = 0) -> torch.Tensor:
    """fp32 score vectors for the selection tests.

    kind: "uniform" U(0,1); "zipf" 1/(rank+1) in a random order (peaked, like
    real attention mass); "flat" 1 + small noise (what random weights give).
    ties > 0 quantises to that many distinct levels to force equal keys.
    """
    g = _gen(seed)
    if kind == "uniform":
        s = torch.rand(n, generator=g)
    elif kind == "zipf":
        s = 1.0 / (1.0 + torch.randperm(n, generator=g).float())
    elif kind == "flat":
        s = 1.0 + 0.05 * torch.randn(n, generator=g).clamp(-3, 3)
    else:
        raise ValueError(kind)
    if ties > 0:
        s = torch.floor(s * ties) / ties
    return s.float()
