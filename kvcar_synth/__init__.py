"""Seeded synthetic inputs for the KV-CAR decode hot path.

This module only *draws numbers* and describes workload shapes.  It holds none of
the method's arithmetic (no encoder, decoder, attention, reuse resolution or page
indexing): both the CPU oracle's tests and the CUDA path's tests/bench are fed
from here, and neither of those two imports the other.

Random streams are counter-based (numpy Philox) and keyed by
``(seed, stream-id words...)`` so that any tensor can be regenerated on its own,
in any order, on any machine.

Workload shapes follow the paper's two evaluation models (a GPT-2-small-shaped
stack: 12 layers x 12 heads x 64; a TinyLLaMA-1.1B-shaped GQA stack: 22 layers,
32 query heads, 4 KV heads x 64) with the autoencoder halving the K/V width
(Table 2: "compressing the key and value vectors by a factor of two").
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

HEAD_DIM = 64


# --------------------------------------------------------------------------
# random streams
# --------------------------------------------------------------------------
def _stream_words(stream) -> List[int]:
    words = []
    for s in stream:
        if isinstance(s, str):
            words.append(zlib.crc32(s.encode()) & 0xFFFFFFFF)
        else:
            words.append(int(s) & 0xFFFFFFFF)
    return words


def rng(seed: int, *stream) -> np.random.Generator:
    """Counter-based generator keyed by (seed, stream words)."""
    words = _stream_words(stream)
    # fold the stream words into a 2x64-bit Philox key, order-sensitively
    k0 = (int(seed) & 0xFFFFFFFF) | (0x9E3779B9 << 32)
    k1 = 0xD1B54A32D192ED03
    for w in words:
        k1 = ((k1 * 6364136223846793005) + w + 1442695040888963407) & 0xFFFFFFFFFFFFFFFF
    return np.random.Generator(np.random.Philox(key=np.array([k0, k1], dtype=np.uint64)))


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16-representable value (ties to
    even) and return them as float32.  Used so that every consumer of a bf16
    workload sees exactly the same input values."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    bias = ((u >> 16) & 1) + 0x7FFF
    u = ((u + bias) >> 16) << 16
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def on_grid(x: np.ndarray, storage: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return to_bf16_grid(x) if storage == "bf16" else x


def normal(shape, seed: int, *stream, storage: str = "f32", scale: float = 1.0) -> np.ndarray:
    g = rng(seed, *stream)
    x = g.standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        x = x * np.float32(scale)
    return on_grid(x, storage)


# --------------------------------------------------------------------------
# workload descriptions (the benchmark configurations)
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    latent_full: int           # latent width of a full-width (no reuse) K or V autoencoder
    batch: int
    cached_tokens: int
    decode_steps: int
    storage: str               # "f32" | "bf16"
    seed: int
    reuse_frac: float
    page_tokens: int = 64
    head_dim: int = HEAD_DIM

    @property
    def kv_width(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def latent_per_head(self) -> int:
        return self.latent_full // self.n_kv_heads

    def pages_per_seq(self) -> int:
        total = self.cached_tokens + self.decode_steps
        return (total + self.page_tokens - 1) // self.page_tokens


CONFIGS: Dict[str, Workload] = {
    # single GPT-2-small-shaped attention layer, fp32, no reuse
    "c1": Workload("c1_gpt2s_1layer_f32", 1, 12, 12, 384, 1, 128, 1, "f32", 0, 0.0),
    # GPT-2-small-shaped full stack
    "c2": Workload("c2_gpt2s_12l_b8_L1024", 12, 12, 12, 384, 8, 1024, 16, "bf16", 1, 0.25),
    # TinyLLaMA-1.1B-shaped GQA stack
    "c3": Workload("c3_tinyllama_22l_b32_L2048", 22, 32, 4, 128, 32, 2048, 64, "bf16", 2, 0.20),
    # TinyLLaMA-shaped long context
    "c4": Workload("c4_tinyllama_22l_b4_L32768", 22, 32, 4, 128, 4, 32768, 8, "bf16", 3, 0.20),
    # GPT-2-small-shaped batch sweep (batch is overridden by the caller)
    "c5": Workload("c5_gpt2s_12l_L4096", 12, 12, 12, 384, 8, 4096, 4, "bf16", 4, 0.25),
}


def with_batch(w: Workload, batch: int) -> Workload:
    return replace(w, batch=batch, name=f"{w.name}_b{batch}")


def scaled(w: Workload, **kw) -> Workload:
    """A smaller/larger variant of a workload (same shapes, other sizes)."""
    return replace(w, **kw)


# --------------------------------------------------------------------------
# reuse maps
# --------------------------------------------------------------------------
def make_reuse_map(n_layers: int, n_kv_heads: int, frac: float, seed: int) -> np.ndarray:
    """Seeded choice of heads in layers >= 1 that point at the same head index of
    the layer below.  Returns int32 [n_layers * n_kv_heads]; -1 = the head stores
    its own data, else the head index in layer l-1.

    Candidates are the (layer >= 1, head) pairs in row-major order; a
    Fisher-Yates shuffle driven by the seeded stream orders them and the first
    round_half_up(frac * count) are taken.
    """
    src = np.full(n_layers * n_kv_heads, -1, dtype=np.int32)
    cand = [(l, h) for l in range(1, n_layers) for h in range(n_kv_heads)]
    n_take = int(np.floor(frac * len(cand) + 0.5))
    if n_take == 0:
        return src
    g = rng(seed, "reuse_map")
    order = list(range(len(cand)))
    for i in range(len(order) - 1, 0, -1):
        j = int(g.integers(0, i + 1))
        order[i], order[j] = order[j], order[i]
    for idx in order[:n_take]:
        l, h = cand[idx]
        src[l * n_kv_heads + h] = h
    return src


def stored_heads(src: np.ndarray, n_kv_heads: int, layer: int) -> List[int]:
    """Heads of `layer` that keep their own cache rows, ascending."""
    row = src[layer * n_kv_heads:(layer + 1) * n_kv_heads]
    return [h for h in range(n_kv_heads) if row[h] < 0]


# --------------------------------------------------------------------------
# autoencoder parameters
# --------------------------------------------------------------------------
def ae_dims(n_stored: int, head_dim: int, latent_per_head: int) -> Tuple[int, int, int]:
    """(in_dim, hidden, latent) of the autoencoder of a layer that stores
    `n_stored` heads: the autoencoder spans only the stored heads, the latent
    keeps the configured ratio, the hidden width is the mean of the two."""
    in_dim = n_stored * head_dim
    latent = n_stored * latent_per_head
    hidden = (in_dim + latent) // 2
    return in_dim, hidden, latent


def _xavier(g: np.random.Generator, fan_out: int, fan_in: int) -> np.ndarray:
    a = np.sqrt(6.0 / (fan_in + fan_out))
    return g.uniform(-a, a, size=(fan_out, fan_in)).astype(np.float32)


def _bias(g: np.random.Generator, fan_out: int, fan_in: int) -> np.ndarray:
    a = 1.0 / np.sqrt(fan_in)
    return g.uniform(-a, a, size=(fan_out,)).astype(np.float32)


def _bn(g: np.random.Generator, n: int, trivial: bool) -> np.ndarray:
    """[4, n] = gamma, beta, running mean, running variance."""
    if trivial:
        return np.stack([np.ones(n), np.zeros(n), np.zeros(n), np.ones(n)]).astype(np.float32)
    gamma = g.uniform(0.5, 1.5, size=n)
    beta = g.standard_normal(n) * 0.1
    mean = g.standard_normal(n) * 0.1
    var = g.uniform(0.5, 1.5, size=n)
    return np.stack([gamma, beta, mean, var]).astype(np.float32)


def make_autoencoder(in_dim: int, hidden: int, latent: int, seed: int, layer: int, which: int,
                     storage: str = "f32", leaky_slope: float = 0.01, bn_eps: float = 1e-5,
                     trivial_bn: bool = False) -> dict:
    """Random-init autoencoder for one (layer, K-or-V).

    Draw order within the stream (seed, "ae", layer, which): encoder W1, b1, BN,
    W2, b2, then decoder W1, b1, BN, W2, b2.  Weights are Xavier-uniform, biases
    U(+-1/sqrt(fan_in)).  Matrices are row-major [out][in].  For bf16 workloads
    the four weight matrices are put on the bf16 grid here (biases and BN
    parameters stay float32; they are applied in fp32 by every consumer).
    """
    g = rng(seed, "ae", layer, which)
    ae = {"in_dim": in_dim, "hidden": hidden, "latent": latent,
          "leaky_slope": float(leaky_slope), "bn_eps": float(bn_eps)}
    ae["enc_w1"] = on_grid(_xavier(g, hidden, in_dim), storage)
    ae["enc_b1"] = _bias(g, hidden, in_dim)
    ae["enc_bn"] = _bn(g, hidden, trivial_bn)
    ae["enc_w2"] = on_grid(_xavier(g, latent, hidden), storage)
    ae["enc_b2"] = _bias(g, latent, hidden)
    ae["dec_w1"] = on_grid(_xavier(g, hidden, latent), storage)
    ae["dec_b1"] = _bias(g, hidden, latent)
    ae["dec_bn"] = _bn(g, hidden, trivial_bn)
    ae["dec_w2"] = on_grid(_xavier(g, in_dim, hidden), storage)
    ae["dec_b2"] = _bias(g, in_dim, hidden)
    return ae


def make_stack_autoencoders(w: Workload, src_k: np.ndarray, src_v: np.ndarray,
                            layers: Optional[List[int]] = None, **kw) -> Dict[Tuple[int, int], dict]:
    """Autoencoders for every (layer, which) of a workload that stores at least
    one head; `layers` restricts compression to some layers (the others keep raw
    K/V, as in the paper's "N layers" rows of Table 2)."""
    out = {}
    for l in range(w.n_layers):
        if layers is not None and l not in layers:
            continue
        for which, src in ((0, src_k), (1, src_v)):
            n = len(stored_heads(src, w.n_kv_heads, l))
            if n == 0:
                continue
            in_dim, hidden, latent = ae_dims(n, w.head_dim, w.latent_per_head)
            out[(l, which)] = make_autoencoder(in_dim, hidden, latent, w.seed, l, which,
                                               storage=w.storage, **kw)
    return out


# --------------------------------------------------------------------------
# activations
# --------------------------------------------------------------------------
def make_kv(w: Workload, layer: int, which: int, seq: int, t0: int, n_tokens: int) -> np.ndarray:
    """Pre-compression K (which=0) or V (which=1) rows of one sequence, tokens
    t0 .. t0+n_tokens-1, [n_tokens, kv_width], ~N(0,1) on the storage grid.
    Generated in blocks of 256 tokens so that any token range is reproducible."""
    blk = 256
    out = np.empty((n_tokens, w.kv_width), dtype=np.float32)
    t = t0
    while t < t0 + n_tokens:
        b = t // blk
        full = normal((blk, w.kv_width), w.seed, "kv", layer, which, seq, b, storage=w.storage)
        lo = t - b * blk
        hi = min(blk, t0 + n_tokens - b * blk)
        out[t - t0:t - t0 + (hi - lo)] = full[lo:hi]
        t += hi - lo
    return out


def make_q(w: Workload, layer: int, seq: int, step: int, scale: float = 1.0) -> np.ndarray:
    """Query of one decode step, [n_q_heads, head_dim], ~N(0,1)*scale."""
    return normal((w.n_q_heads, w.head_dim), w.seed, "q", layer, seq, step,
                  storage=w.storage, scale=scale)
