"""Seeded synthetic inputs for the quantized-forward path.

This module only draws random tensors and routing tables; it holds none of the
method's arithmetic (no quantization, no GEMM, no SwiGLU, no combine).  Both the
CPU oracle's tests and the CUDA path's tests take their inputs from here so that
the two sides see identical bytes.

All tensors are returned as numpy arrays.  bf16 tensors are returned as
``uint16`` arrays holding the bf16 bit patterns (numpy has no bf16); the
conversion fp32 -> bf16 uses torch's CPU cast (round to nearest even).

Shapes follow the Qwen3-30B-A3B-shaped workloads: hidden H = 2048, MoE
intermediate I = 768, E = 128 experts, top-k = 8, QKV projection N = 5120.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

H_QWEN3 = 2048
I_QWEN3 = 768
E_QWEN3 = 128
TOPK_QWEN3 = 8
N_QKV_QWEN3 = 5120


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 array -> uint16 array of bf16 bit patterns (round to nearest even)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """uint16 array of bf16 bit patterns -> fp32 array (exact)."""
    return (b.astype(np.uint32) << 16).view(np.float32)


def weight_bf16(rng: np.random.Generator, *shape: int, std: float = 0.02) -> np.ndarray:
    """W ~ N(0, std^2), rounded to bf16."""
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))


def act_bf16(rng: np.random.Generator, m: int, k: int, outlier_frac: float = 0.01,
             outlier_gain: float = 50.0) -> np.ndarray:
    """X ~ N(0, 1) with a fraction of entries multiplied by a gain (activation
    outliers), rounded to bf16."""
    x = rng.standard_normal((m, k), dtype=np.float32)
    if outlier_frac > 0:
        mask = rng.random((m, k)) < outlier_frac
        x = np.where(mask, x * np.float32(outlier_gain), x)
    return f32_to_bf16_bits(x)


def zipf_log_popularity(rng: np.random.Generator, e: int, s: float = 1.1) -> np.ndarray:
    """ln p_e with p_e proportional to rank_e^(-s), rank a random permutation of 1..E."""
    rank = rng.permutation(e).astype(np.float64) + 1.0
    p = rank ** (-s)
    p /= p.sum()
    return np.log(p)


def routing(rng: np.random.Generator, m: int, e: int, k: int,
            log_popularity: np.ndarray | None = None) -> tuple[np.ndarray, np.ndarray]:
    """Draw router logits ~ N(0,1) (+ optional per-expert bias), take the top-k
    experts per token (ties to the lower expert id) and weight them by a softmax
    over the k selected logits.  Returns (ids int32 [m,k], weights fp32 [m,k]).
    The k slots of a token are in descending-logit order, i.e. NOT sorted by
    expert id, as a router would emit them."""
    logits = rng.standard_normal((m, e))
    if log_popularity is not None:
        logits = logits + log_popularity[None, :]
    # stable argsort of -logits: ties resolve to the lower expert id
    order = np.argsort(-logits, axis=1, kind="stable")[:, :k]
    sel = np.take_along_axis(logits, order, axis=1)
    sel = sel - sel.max(axis=1, keepdims=True)
    w = np.exp(sel)
    w /= w.sum(axis=1, keepdims=True)
    return order.astype(np.int32), w.astype(np.float32)


@dataclass
class LinearCase:
    w: np.ndarray   # bf16 bits [N, K]
    x: np.ndarray   # bf16 bits [M, K]
    M: int
    N: int
    K: int


def linear_case(seed: int, m: int, n: int, k: int) -> LinearCase:
    rng = np.random.default_rng(seed)
    w = weight_bf16(rng, n, k)
    x = act_bf16(rng, m, k)
    return LinearCase(w=w, x=x, M=m, N=n, K=k)


def config1() -> LinearCase:
    """Single quantized linear, seed 0: W [256, 512], X [16, 512]."""
    return linear_case(0, 16, 256, 512)


def config2(m: int) -> LinearCase:
    """Dense QKV projection K = 2048, N = 5120 at M = 64 (decode) or 8192 (train)."""
    return linear_case(2, m, N_QKV_QWEN3, H_QWEN3)


@dataclass
class MoeCase:
    x: np.ndarray        # bf16 bits [M, H]
    w13: np.ndarray      # bf16 bits [E, 2I, H]; rows 0..I-1 gate, I..2I-1 up
    w2: np.ndarray       # bf16 bits [E, H, I]
    ids: np.ndarray      # int32 [M, k]
    weights: np.ndarray  # fp32 [M, k]
    M: int
    H: int
    I: int
    E: int
    k: int


def moe_case(seed: int, m: int, h: int = H_QWEN3, i: int = I_QWEN3, e: int = E_QWEN3,
             k: int = TOPK_QWEN3, zipf_s: float | None = None) -> MoeCase:
    """One MoE FFN layer.  zipf_s=None: unbiased router (decode shape);
    zipf_s=1.1: expert popularity follows Zipf(s) (training shape)."""
    rng = np.random.default_rng(seed)
    w13 = weight_bf16(rng, e, 2 * i, h)
    w2 = weight_bf16(rng, e, h, i)
    x = act_bf16(rng, m, h)
    logp = zipf_log_popularity(rng, e, zipf_s) if zipf_s is not None else None
    ids, wts = routing(rng, m, e, k, logp)
    return MoeCase(x=x, w13=w13, w2=w2, ids=ids, weights=wts, M=m, H=h, I=i, E=e, k=k)


def config3() -> MoeCase:
    """MoE FFN layer at decode: M = 256, unbiased router."""
    return moe_case(3, 256)


def config4(m: int = 32768) -> MoeCase:
    """MoE FFN layer at the training-forward shape: M = 32768, Zipf(1.1) popularity."""
    return moe_case(4, m, zipf_s=1.1)


# --------------------------------------------------------------------------- TBPO loss inputs
def tbpo_case(seed: int, lengths, drift: float = 5e-4, mismatch: float = 0.02):
    """Packed per-token log-probs of B responses with the given lengths (a list/array of ints,
    zeros allowed): the old sampler's (negative, heavy towards small magnitudes), the old
    learner's = sampler + N(0, mismatch) (quantized-rollout mismatch), the current learner's =
    old learner + a per-response shift N(0, drift) + token noise N(0, 2 drift) (one optimizer
    step away, so that the sequence ratios straddle the 1e-3-wide trust bands), and
    group-normalized-looking advantages N(0, 1).  Returns fp32 arrays and int64 offsets."""
    rng = np.random.default_rng(seed)
    lengths = np.asarray(lengths, dtype=np.int64)
    off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    T = int(off[-1])
    smp = (-np.abs(rng.normal(0.0, 1.5, size=T)) - 0.01).astype(np.float32)
    old = (smp + rng.normal(0.0, mismatch, size=T)).astype(np.float32)
    shift = np.repeat(rng.normal(0.0, drift, size=len(lengths)), lengths)
    cur = (old + shift + rng.normal(0.0, 2 * drift, size=T)).astype(np.float32)
    adv = rng.normal(0.0, 1.0, size=len(lengths)).astype(np.float32)
    return cur, old, smp, off, adv


def tbpo_lengths(seed: int, b: int, mean_len: int = 4096, max_len: int = 16384) -> np.ndarray:
    """Response lengths: lognormal around mean_len (sigma 0.8), clipped to [16, max_len]."""
    rng = np.random.default_rng(seed)
    l = rng.lognormal(np.log(mean_len) - 0.32, 0.8, size=b)
    return np.clip(l, 16, max_len).astype(np.int64)
