"""Seeded synthetic workloads: shapes, lengths, layer masks and N(0,1) bf16 tensors.

This module only draws numbers and describes shapes.  It holds none of the
attention arithmetic and is the one module both the CUDA tests/benchmark and
the CPU oracle's callers take inputs from; the same bits are handed to both
sides.  The shapes are the attention stacks of the backbones the paper
evaluates (Sec. 4.1: Llama-3.1-8B is 32 layers, 32 query / 8 KV heads, head
dim 128) with the kernel constants of its Sparsity Config (Table 3: sink 128,
local 2048, block 64, chunk 16384); benchmark prompts are replaced by i.i.d.
N(0,1) values rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

MASTER_SEED = 0xF1A70000


@dataclass(frozen=True)
class Workload:
    """One synthetic configuration of the routed attention stack."""

    name: str
    cfg_id: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    batch: int
    sink: int
    window: int
    prompt_len: int          # tokens prefilled (0 if the workload starts from a given cache)
    ctx_lo: int              # context length(s) the decode phase starts from
    ctx_hi: int
    decode_steps: int
    mask_rule: str           # "fixed" | "bernoulli" | "exact" | "fraction"
    mask_arg: tuple = field(default_factory=tuple)

    @property
    def seed(self) -> int:
        return MASTER_SEED + self.cfg_id


WORKLOADS = {
    # correctness configuration: everything small enough for a full oracle sweep
    "cfg1": Workload("cfg1", 1, 4, 8, 2, 128, 1, 64, 256, 1024, 1024, 1024, 16, "fixed", (1, 0, 1, 0)),
    # long prefill, Llama-3-8B attention shapes
    "cfg2": Workload("cfg2", 2, 32, 32, 8, 128, 1, 128, 2048, 32768, 32768, 32768, 0, "bernoulli", (0.5,)),
    # batched long-context decode
    "cfg3": Workload("cfg3", 3, 32, 32, 8, 128, 8, 128, 4096, 0, 65536, 65536, 256, "exact", (0.5,)),
    # 128K prefill then decode, G = 7
    "cfg4": Workload("cfg4", 4, 28, 28, 4, 128, 1, 128, 4096, 131072, 131072, 131072, 128, "exact", (0.75,)),
    # ragged mixed-routing decode
    "cfg5": Workload("cfg5", 5, 32, 32, 8, 128, 16, 128, 4096, 0, 4096, 131072, 128, "fraction", (0.25, 0.9)),
}


def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.default_rng([seed & 0xFFFFFFFF, *[int(s) & 0xFFFFFFFF for s in stream]])


def layer_masks(w: Workload) -> np.ndarray:
    """Per-request layer masks ``[B][L]`` uint8, 1 = FA, 0 = SA (Sec. 3.1 encoding)."""
    B, L = w.batch, w.n_layers
    rng = _rng(w.seed, 1)
    mask = np.ones((B, L), dtype=np.uint8)
    if w.mask_rule == "fixed":
        mask[:] = np.asarray(w.mask_arg, dtype=np.uint8)[None, :]
    elif w.mask_rule == "bernoulli":
        mask[:] = (rng.random((B, L)) >= w.mask_arg[0]).astype(np.uint8)
    elif w.mask_rule == "exact":
        n_sa = int(round(w.mask_arg[0] * L))
        for b in range(B):
            mask[b, rng.permutation(L)[:n_sa]] = 0
    elif w.mask_rule == "fraction":
        lo, hi = w.mask_arg
        for b in range(B):
            n_sa = int(round(L * rng.uniform(lo, hi)))
            mask[b, rng.permutation(L)[:n_sa]] = 0
    else:
        raise ValueError(w.mask_rule)
    return mask


def masks_to_logits(mask: np.ndarray, seed: int) -> np.ndarray:
    """Routing logits ``[B][L][2]`` fp32 (FA first) whose argmax reproduces ``mask``."""
    rng = _rng(seed, 2)
    B, L = mask.shape
    hi = rng.uniform(0.5, 3.0, size=(B, L)).astype(np.float32)
    lo = hi - rng.uniform(0.1, 2.0, size=(B, L)).astype(np.float32)
    lg = np.empty((B, L, 2), dtype=np.float32)
    lg[..., 0] = np.where(mask == 1, hi, lo)
    lg[..., 1] = np.where(mask == 1, lo, hi)
    return lg


def context_lengths(w: Workload) -> np.ndarray:
    """Context length per request at the start of decode, ``[B]`` int32."""
    if w.ctx_lo == w.ctx_hi:
        return np.full(w.batch, w.ctx_lo, dtype=np.int32)
    rng = _rng(w.seed, 3)
    u = rng.uniform(np.log(w.ctx_lo), np.log(w.ctx_hi), size=w.batch)
    return np.clip(np.rint(np.exp(u)), w.ctx_lo, w.ctx_hi).astype(np.int32)


def _mix(seed: int, stream: int) -> int:
    return ((int(seed) & 0xFFFFFFFF) * 0x100000000 + (int(stream) & 0xFFFFFFFF)) & 0x7FFFFFFFFFFFFFFF


def normal_bf16(shape, seed: int, stream: int, device="cpu") -> torch.Tensor:
    """i.i.d. N(0,1) values rounded to bf16; one generator stream per (seed, stream)."""
    g = torch.Generator(device=device)
    g.manual_seed(_mix(seed, stream))
    t = torch.empty(shape, dtype=torch.bfloat16, device=device)
    t.normal_(0.0, 1.0, generator=g)
    return t


def fill_normal_bf16_(t: torch.Tensor, seed: int, stream: int) -> torch.Tensor:
    """In-place variant of :func:`normal_bf16` for buffers that are already allocated."""
    g = torch.Generator(device=t.device)
    g.manual_seed(_mix(seed, stream))
    t.normal_(0.0, 1.0, generator=g)
    return t


# stream ids: tensor kind * 2^12 + layer * 2^6 ... kept simple and collision-free
def stream_id(kind: str, layer: int = 0, req: int = 0, step: int = 0) -> int:
    kinds = {"q": 1, "k": 2, "v": 3, "qdec": 4, "kdec": 5, "vdec": 6, "router": 7}
    return ((kinds[kind] * 64 + layer) * 64 + req) * 1024 + step


def router_weights(seed: int, layer: int, n_features: int, enc_dim: int, head_hidden: int, device="cpu") -> dict:
    """Random stand-ins for one layer's trained router (Sec. 3.1): bf16 weight matrices with
    N(0, 1/fan_in) entries and fp32 biases N(0, 0.1^2), so every layer's outputs stay O(1).
    Keys: w_enc1 [E][F], w_enc2 [E][E], w_head1 [R][E], w_head2 [2][R], b_enc1, b_enc2, b_head1,
    b_head2.  Drawn on the CPU (the same bits whatever the device) and moved."""
    shapes = {"w_enc1": (enc_dim, n_features), "w_enc2": (enc_dim, enc_dim),
              "w_head1": (head_hidden, enc_dim), "w_head2": (2, head_hidden)}
    out = {}
    for step, (name, shp) in enumerate(shapes.items()):
        g = torch.Generator(device="cpu")
        g.manual_seed(_mix(seed, stream_id("router", layer, 0, step)))
        w = torch.empty(shp, dtype=torch.float32).normal_(0.0, 1.0, generator=g) / float(np.sqrt(shp[1]))
        out[name] = w.to(torch.bfloat16).to(device)
        b = torch.empty(shp[0], dtype=torch.float32).normal_(0.0, 0.1, generator=g)
        out[name.replace("w_", "b_")] = b.to(device)
    return out


def sample_rows(n_rows_total: int, sink: int, window: int, n_random: int, seed: int,
                q_start: int = 0) -> np.ndarray:
    """Query positions for sampled parity checks: set boundaries, tile edges, random rows."""
    N = q_start + n_rows_total
    S, W = sink, window
    cand = [0, 1, S - 1, S, S + 1, W - 1, W, S + W - 2, S + W - 1, S + W, S + W + 1,
            63, 64, 127, 128, 129, 255, 256, N // 2 - 1, N // 2, N - 129, N - 128, N - 2, N - 1]
    rng = _rng(seed, 4)
    cand += list(rng.integers(q_start, N, size=n_random))
    rows = sorted({int(c) for c in cand if q_start <= c < N})
    return np.asarray(rows, dtype=np.int64)
