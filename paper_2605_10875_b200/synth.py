"""Seeded synthetic workloads for the action-conditioned decode step.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic, so both the CPU oracle's tests and the CUDA path may be
fed from it.  Everything is NumPy; bf16 tensors are uint16 bit patterns.

The five workloads follow the task's configurations: weights ~ N(0, 0.02),
KV cache and hidden state ~ N(0, 1), RMSNorm gains ~ 1 + N(0, 0.02), a paged
cache of 64-token pages with a shuffled page table (identity for the
contiguous tiny case), and per-sequence actions drawn uniformly from small
value sets.  They stand in for real activations of a Llama-shaped model; no
dataset or checkpoint is involved.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np

WORKLOADS: Dict[str, dict] = {
    # 1: tiny single decoder layer, contiguous 512-token cache
    "tiny": dict(layers=1, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ff=1024, batch=4,
                 context=512, rope_theta=0.0, shuffle_pages=False,
                 r_set=(250, 500, 1000), p_set=(0, 250, 500), b_set=(4, 8, 16)),
    # 2: one Llama-3.2-1B-shaped layer
    "llama1b_layer": dict(layers=1, d_model=2048, n_q_heads=32, n_kv_heads=8, head_dim=64, d_ff=8192, batch=16,
                          context=4096, rope_theta=500000.0, shuffle_pages=True,
                          r_set=(125, 250, 500, 1000), p_set=(0, 250, 500, 750), b_set=(4, 8, 16)),
    # 3: 16 layers of the same shape
    "llama1b_step": dict(layers=16, d_model=2048, n_q_heads=32, n_kv_heads=8, head_dim=64, d_ff=8192, batch=32,
                         context=8192, rope_theta=500000.0, shuffle_pages=True,
                         r_set=(125, 250, 500, 1000), p_set=(0, 250, 500, 750), b_set=(4, 8, 16)),
    # 4: one Llama-3.1-8B-shaped layer
    "llama8b_layer": dict(layers=1, d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ff=14336, batch=64,
                          context=16384, rope_theta=500000.0, shuffle_pages=True,
                          r_set=(125, 250, 500, 1000), p_set=(0, 250, 500, 750), b_set=(4, 8, 16)),
    # 5: ragged serving mix, lognormal contexts (median 4096, sigma 1 in log space) clipped to [256, 32768]
    "ragged_serving": dict(layers=16, d_model=2048, n_q_heads=32, n_kv_heads=8, head_dim=64, d_ff=8192, batch=128,
                           context=None, context_median=4096, context_sigma=1.0, context_clip=(256, 32768),
                           rope_theta=500000.0, shuffle_pages=True,
                           r_set=(125, 250, 500, 1000), p_set=(0, 250, 500, 750), b_set=(4, 8, 16)),
}

PAGE_SIZE = 64
RMS_EPS = 1e-5

_STREAMS = dict(w_qkv=1, w_o=2, w_gate=3, w_up=4, w_down_t=5, gamma1=6, gamma2=7, k_pool=8, v_pool=9,
                hidden=10, actions=11, pages=12, contexts=13, q=14)


def rng_for(seed: int, stream: str, layer: int = 0, extra: int = 0) -> np.random.Generator:
    """An independent generator per (seed, named tensor, layer)."""
    return np.random.default_rng([int(seed), _STREAMS[stream], int(layer), int(extra)])


def to_bf16(x32: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round-to-nearest-even (input preparation)."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(u16: np.ndarray) -> np.ndarray:
    return (np.asarray(u16, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, mean: float, std: float, chunk: int = 1 << 24) -> np.ndarray:
    """N(mean, std) rounded to bf16, generated in chunks to bound host memory."""
    n = int(np.prod(shape))
    out = np.empty(n, np.uint16)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = rng.standard_normal(e - s, dtype=np.float32)
        x *= np.float32(std)
        if mean:
            x += np.float32(mean)
        out[s:e] = to_bf16(x)
    return out.reshape(shape)


@dataclass
class LayerTensors:
    w_qkv: np.ndarray
    w_o: np.ndarray
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down_t: np.ndarray
    gamma1: np.ndarray
    gamma2: np.ndarray


def make_layer_weights(cfg: dict, seed: int = 0, layer: int = 0) -> LayerTensors:
    d, hq, hkv, hd, ff = cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_ff"]
    g = lambda name: rng_for(seed, name, layer)
    return LayerTensors(
        w_qkv=normal_bf16(g("w_qkv"), ((hq + 2 * hkv) * hd, d), 0.0, 0.02),
        w_o=normal_bf16(g("w_o"), (d, hq * hd), 0.0, 0.02),
        w_gate=normal_bf16(g("w_gate"), (ff, d), 0.0, 0.02),
        w_up=normal_bf16(g("w_up"), (ff, d), 0.0, 0.02),
        w_down_t=normal_bf16(g("w_down_t"), (ff, d), 0.0, 0.02),
        gamma1=normal_bf16(g("gamma1"), (d,), 1.0, 0.02),
        gamma2=normal_bf16(g("gamma2"), (d,), 1.0, 0.02),
    )


def make_contexts(cfg: dict, seed: int = 0, batch: Optional[int] = None) -> np.ndarray:
    """Per-sequence context lengths (tokens in the cache INCLUDING the newest)."""
    B = batch or cfg["batch"]
    if cfg.get("context") is not None:
        return np.full(B, cfg["context"], np.int32)
    rng = rng_for(seed, "contexts")
    lo, hi = cfg["context_clip"]
    t = np.exp(np.log(cfg["context_median"]) + cfg["context_sigma"] * rng.standard_normal(B))
    return np.clip(np.rint(t), lo, hi).astype(np.int32)


def make_page_table(seq_lens: np.ndarray, shuffle: bool, seed: int = 0, spare_tokens: int = 0
                    ) -> Tuple[np.ndarray, int]:
    """Assign physical pages.  Returns (page_table [B][max_pages], num_pages).
    spare_tokens reserves room per sequence for later appends.  Unused table
    entries are -1."""
    B = len(seq_lens)
    need = [(int(t) + spare_tokens + PAGE_SIZE - 1) // PAGE_SIZE for t in seq_lens]
    num_pages = int(sum(need))
    ids = np.arange(num_pages, dtype=np.int32)
    if shuffle:
        rng_for(seed, "pages").shuffle(ids)
    table = np.full((B, max(need)), -1, np.int32)
    at = 0
    for i, n in enumerate(need):
        table[i, :n] = ids[at:at + n]
        at += n
    return table, num_pages


def make_kv_pool(cfg: dict, num_pages: int, seed: int = 0, layer: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    shape = (num_pages, cfg["n_kv_heads"], PAGE_SIZE, cfg["head_dim"])
    return (normal_bf16(rng_for(seed, "k_pool", layer), shape, 0.0, 1.0),
            normal_bf16(rng_for(seed, "v_pool", layer), shape, 0.0, 1.0))


def device_kv_pool(cfg: dict, num_pages: int, device, seed: int = 0, layer: int = 0):
    """The same N(0, 1) bf16 pools drawn on a CUDA device by torch's counter-based generator, for
    workloads whose cache (tens of GB) would take minutes to draw on the host.  Returns torch bf16
    tensors (k_pool, v_pool); a checker reads back the pages it needs."""
    return (device_normal_bf16((num_pages, cfg["n_kv_heads"], PAGE_SIZE, cfg["head_dim"]), device, seed, "k_pool", layer),
            device_normal_bf16((num_pages, cfg["n_kv_heads"], PAGE_SIZE, cfg["head_dim"]), device, seed, "v_pool", layer))


def device_normal_bf16(shape, device, seed: int, stream: str, layer: int = 0, mean: float = 0.0, std: float = 1.0):
    """N(mean, std) rounded to bf16, drawn on `device` (torch): an independent seeded stream per
    (seed, named tensor, layer), like rng_for."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + _STREAMS[stream]) * 1000003 + int(layer))
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    chunk = 1 << 28
    for s0 in range(0, flat.numel(), chunk):
        part = flat[s0:s0 + chunk]
        x = torch.randn(part.shape, dtype=torch.float32, device=device, generator=g)
        part.copy_(x.mul_(std).add_(mean))
    return out


def device_layer_weights(cfg: dict, device, seed: int = 0, layer: int = 0) -> dict:
    """Layer weights of the workload's shapes and distributions drawn on the device (see device_normal_bf16)."""
    d, hq, hkv, hd, ff = cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["d_ff"]
    g = lambda name, shape, mean, std: device_normal_bf16(shape, device, seed, name, layer, mean, std)
    return dict(w_qkv=g("w_qkv", ((hq + 2 * hkv) * hd, d), 0.0, 0.02), w_o=g("w_o", (d, hq * hd), 0.0, 0.02),
                w_gate=g("w_gate", (ff, d), 0.0, 0.02), w_up=g("w_up", (ff, d), 0.0, 0.02),
                w_down_t=g("w_down_t", (ff, d), 0.0, 0.02), gamma1=g("gamma1", (d,), 1.0, 0.02),
                gamma2=g("gamma2", (d,), 1.0, 0.02))


def make_hidden(cfg: dict, seed: int = 0, batch: Optional[int] = None) -> np.ndarray:
    B = batch or cfg["batch"]
    return normal_bf16(rng_for(seed, "hidden"), (B, cfg["d_model"]), 0.0, 1.0)


def make_queries(cfg: dict, seed: int = 0, batch: Optional[int] = None) -> np.ndarray:
    """bf16 queries for the stand-alone attention call, N(0, 1)."""
    B = batch or cfg["batch"]
    return normal_bf16(rng_for(seed, "q"), (B, cfg["n_q_heads"], cfg["head_dim"]), 0.0, 1.0)


def draw_actions(cfg: dict, seed: int = 0, batch: Optional[int] = None, redraw: int = 0):
    """Per-sequence (r_permille, p_permille, bits), uniform over the value sets."""
    B = batch or cfg["batch"]
    rng = rng_for(seed, "actions", 0, redraw)
    pick = lambda vals: np.asarray(vals, np.int32)[rng.integers(0, len(vals), B)]
    return pick(cfg["r_set"]), pick(cfg["p_set"]), pick(cfg["b_set"])


def uniform_actions(batch: int, r_permille: int, p_permille: int, bits: int):
    """Every sequence with the same action: one point of a budget sweep."""
    f = lambda v: np.full(batch, v, np.int32)
    return f(r_permille), f(p_permille), f(bits)


def budget_mix_actions(cfg: dict, target_permille: int, seed: int = 0, batch: Optional[int] = None):
    """Actions whose batch-mean r*(1-p) hits a target, by mixing the two
    adjacent levels of the r grid across the batch with p = 0 (how the paper's
    fixed baseline matches a budget that falls between discrete levels).
    Bit-widths are drawn uniformly.  target 1000 gives r = 1, p = 0 everywhere."""
    B = batch or cfg["batch"]
    levels = sorted(cfg["r_set"])
    rng = rng_for(seed, "actions", 0, 10_000 + target_permille)
    bits = np.asarray(cfg["b_set"], np.int32)[rng.integers(0, len(cfg["b_set"]), B)]
    p = np.zeros(B, np.int32)
    tgt = min(max(target_permille, levels[0]), levels[-1])
    hi = next(v for v in levels if v >= tgt)
    lo = max([v for v in levels if v <= tgt])
    n_hi = B if hi == lo else int(round(B * (tgt - lo) / (hi - lo)))
    r = np.full(B, lo, np.int32)
    r[rng.permutation(B)[:n_hi]] = hi
    return r, p, bits
