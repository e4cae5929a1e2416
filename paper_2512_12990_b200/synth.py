"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers.  It holds none of the method's arithmetic (no
quantiser, no slicing, no routing, no FFN): both the CPU oracle's tests and the
CUDA path's tests/bench take their inputs from here so that the two sides see
identical bits, and neither side's code is involved in producing them.

Every stream is a counter-based Philox generator keyed by (seed, stream id), so
any array can be regenerated on its own without generating the ones before it.

The two evaluated models (Section 6.1 of the paper: DeepSeek-V2-Lite and
Qwen1.5-MoE-A2.7B) are represented by their MoE layer *shapes* only; weights are
N(0, 0.02), activations N(0, 1) rounded to bf16, router logits as described per
function.  No model weights and no benchmark items are used.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field

import numpy as np

__all__ = [
    "Shape", "SHAPES", "stream_id", "rng", "normal_f32", "bf16_round", "bf16_to_f32",
    "bf16_to_f64", "activations_bf16", "expert_weights", "router_logits_normal",
    "zipf_gumbel_logits", "decode_trace_logits", "prefill_trace_logits",
]


@dataclass(frozen=True)
class Shape:
    """One MoE layer shape (no arithmetic; just sizes)."""
    name: str
    hidden: int
    inter: int
    n_experts: int
    top_k: int
    group: int
    n_shared: int = 0
    shared_inter: int = 0
    shared_sigmoid_gate: bool = False
    n_layers: int = 1
    seed: int = 0


SHAPES = {
    # tiny single layer: hidden 256, 8 experts x inter 128, top-2, group 64
    "tiny": Shape("tiny", 256, 128, 8, 2, 64, seed=1001),
    # DeepSeek-V2-Lite-shaped: hidden 2048, 64 routed x 1408, top-6, 2 shared x 1408, group 128
    "dsv2": Shape("dsv2", 2048, 1408, 64, 6, 128, n_shared=2, shared_inter=1408, seed=1002),
    # Qwen1.5-MoE-A2.7B-shaped: hidden 2048, 60 routed x 1408, top-4, one shared 5632 with sigmoid gate
    "qwen": Shape("qwen", 2048, 1408, 60, 4, 128, n_shared=1, shared_inter=5632,
                  shared_sigmoid_gate=True, seed=1003),
    # DeepSeek-V2-Lite-shaped decode stack: 26 layers
    "dsv2_stack": Shape("dsv2_stack", 2048, 1408, 64, 6, 128, n_shared=2, shared_inter=1408,
                        n_layers=26, seed=1004),
    # Qwen-shaped prefill layer (2048 tokens)
    "qwen_prefill": Shape("qwen_prefill", 2048, 1408, 60, 4, 128, n_shared=1, shared_inter=5632,
                          shared_sigmoid_gate=True, seed=1005),
}


def stream_id(*parts) -> int:
    """Stable 64-bit id of a named stream, e.g. stream_id("W", layer, expert, "gate")."""
    h = hashlib.blake2b("/".join(str(p) for p in parts).encode(), digest_size=8).digest()
    return int.from_bytes(h, "little")


def rng(seed: int, *parts) -> np.random.Generator:
    """Counter-based generator for one (seed, stream)."""
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), stream_id(*parts)]))


def normal_f32(seed: int, parts, shape, std: float = 1.0) -> np.ndarray:
    """N(0, std^2) as float32."""
    g = rng(seed, *parts)
    a = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def bf16_round(a_f32: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a_f32, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_to_f32(bits_u16: np.ndarray) -> np.ndarray:
    return (bits_u16.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(bits_u16: np.ndarray) -> np.ndarray:
    return bf16_to_f32(bits_u16).astype(np.float64)


def activations_bf16(seed: int, parts, shape) -> np.ndarray:
    """Activations ~ N(0,1) rounded to bf16; returned as uint16 bit patterns."""
    return bf16_round(normal_f32(seed, parts, shape))


def expert_weights(seed: int, layer: int, expert, hidden: int, inter: int, std: float = 0.02):
    """The three fp32 matrices of one SwiGLU expert, row-major [N_out, K_in].

    `expert` is an int for a routed expert or a string such as "shared0".
    Returns dict(gate=[inter, hidden], up=[inter, hidden], down=[hidden, inter]).
    """
    return {
        "gate": normal_f32(seed, ("W", layer, expert, "gate"), (inter, hidden), std),
        "up": normal_f32(seed, ("W", layer, expert, "up"), (inter, hidden), std),
        "down": normal_f32(seed, ("W", layer, expert, "down"), (hidden, inter), std),
    }


def router_logits_normal(seed: int, parts, T: int, E: int) -> np.ndarray:
    """Router logits ~ N(0,1), float32 [T, E]."""
    return normal_f32(seed, parts, (T, E))


def _zipf_logp(E: int, s: float, perm: np.ndarray) -> np.ndarray:
    ranks = np.arange(1, E + 1, dtype=np.float64)
    p = ranks ** (-s)
    p /= p.sum()
    logp = np.empty(E, dtype=np.float64)
    logp[perm] = np.log(p)           # expert perm[r] has popularity rank r
    return logp


def zipf_gumbel_logits(seed: int, parts, T: int, E: int, s: float):
    """Logits = log(popularity) + Gumbel noise, popularity Zipf(s) over a seeded expert
    permutation.  Top-k of such logits samples k experts without replacement in proportion
    to popularity.  Returns (logits float32 [T, E], perm) with perm[r] = expert of rank r."""
    g = rng(seed, *parts)
    perm = g.permutation(E)
    logp = _zipf_logp(E, s, perm)
    u = g.random(size=(T, E), dtype=np.float64)
    u = np.clip(u, 1e-300, 1.0 - 1e-16)
    gumbel = -np.log(-np.log(u))
    return (logp[None, :] + gumbel).astype(np.float32), perm


def decode_trace_logits(seed: int, n_steps: int, n_layers: int, E: int, s: float = 1.1,
                        p_repeat: float = 0.5):
    """Router logits for a decode run: float32 [n_steps, n_layers, E].

    Per layer: Zipf(s) popularity over a seeded permutation plus Gumbel noise per step; with
    probability p_repeat a (step, layer) reuses the previous step's logits of that layer, so
    the same expert set is selected again (temporal reuse)."""
    out = np.empty((n_steps, n_layers, E), dtype=np.float32)
    for l in range(n_layers):
        fresh, _ = zipf_gumbel_logits(seed, ("trace", l), n_steps, E, s)
        g = rng(seed, "trace-repeat", l)
        rep = g.random(n_steps) < p_repeat
        for t in range(n_steps):
            if t > 0 and rep[t]:
                out[t, l] = out[t - 1, l]
            else:
                out[t, l] = fresh[t]
    return out


def prefill_trace_logits(seed: int, n_tokens: int, n_layers: int, E: int, s: float = 1.1) -> np.ndarray:
    """Router logits of a prompt that precedes the decode run of decode_trace_logits: float32
    [n_layers, n_tokens, E].  Per layer the Zipf(s) popularity sits on the SAME expert permutation as
    the decode trace (experts that are hot in prefill stay hot in early decode), the Gumbel noise
    is drawn from a stream of its own."""
    out = np.empty((n_layers, n_tokens, E), dtype=np.float32)
    for l in range(n_layers):
        perm = rng(seed, "trace", l).permutation(E)   # the first draw of the decode trace's stream
        logp = _zipf_logp(E, s, perm)
        u = rng(seed, "prefill-trace", l).random(size=(n_tokens, E), dtype=np.float64)
        u = np.clip(u, 1e-300, 1.0 - 1e-16)
        out[l] = (logp[None, :] - np.log(-np.log(u))).astype(np.float32)
    return out
