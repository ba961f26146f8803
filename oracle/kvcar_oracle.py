"""CPU oracle for the KV-CAR decode hot path.  TEST INFRASTRUCTURE, not product code.

A plain, slow, fp64 numpy statement of what the path computes, written from the
paper's description and sharing nothing with the CUDA library: the encoder that
shrinks a new token's K and V along the embedding dimension and appends the
latent to a cache (Sec. "Network Architecture"), the decoder that restores every
cached row on retrieval, scaled-dot-product attention over the restored rows plus
the exact current token (Eq. 1), and the cross-layer head reuse table (same
section, last paragraph).  Only tests, the smoke check and the benchmark's CPU
baseline may call it.

Parity status: every function here is pinned by special cases, closed forms and
brute force in the CPU test-suite, EXCEPT the numeric value of the nonlinear
autoencoder + attention on the benchmark-sized random inputs, for which the paper
prints no value: that composite is "parity unpinned" beyond those special cases.

Readings of points the paper leaves open are listed in the repository's design
notes; the ones that matter for reading this file:
  * separate autoencoders for K and for V, per layer, spanning the heads that the
    layer stores (a reused head is never encoded or stored);
  * FC -> BatchNorm (inference statistics) -> LeakyReLU -> FC, biases in all FCs,
    nothing after the last FC, for encoder and decoder alike;
  * a head table entry points at a head of layer l-1; chains resolve transitively;
  * cached tokens are attended through their restored rows, the current token
    through its exact K/V (Sec. "Network Architecture": the restored rows are joined with
    the current token's exact key and value vectors).
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

K, V = 0, 1


# --------------------------------------------------------------------------
# storage format
# --------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 value (8 significant bits, ties to even), computed
    directly from fp64 so that no intermediate fp32 rounding interferes."""
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    nz = x != 0
    if np.any(nz):
        mant, exp = np.frexp(x[nz])           # x = mant * 2**exp, 0.5 <= |mant| < 1
        exp = np.maximum(exp, -125)           # bf16 normal range floor (subnormals share one quantum)
        quantum = np.ldexp(1.0, exp - 8)      # spacing of 8-bit significands in that binade
        out[nz] = np.rint(x[nz] / quantum) * quantum
    return out


def round_to_storage(x: np.ndarray, storage: str) -> np.ndarray:
    if storage == "exact":
        return np.asarray(x, dtype=np.float64)
    if storage == "f32":
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
    if storage == "bf16":
        return round_to_bf16(x)
    if storage == "int8":
        return int8_rows(x)
    raise ValueError(storage)


STORAGE_BYTES = {"exact": 8, "f32": 4, "bf16": 2, "int8": 1}
INT8_ROW_PARAM_BYTES = 8   # scale and zero-point (fp32 each) kept beside every int8 row


# --------------------------------------------------------------------------
# Eq. 3 and Eq. 4
# --------------------------------------------------------------------------
def kv_cache_size_bytes(bytes_per_elem: int, n_layers: int, d_model: int, seq_len: int, batch: int) -> int:
    """Eq. 3: 2 x P x N_layers x d_model x L_seq x B."""
    return 2 * bytes_per_elem * n_layers * d_model * seq_len * batch


def int8_quantize(x: np.ndarray) -> Tuple[np.ndarray, float, float]:
    """Eq. 4: scale = 255/(max-min); zeropoint = -round(scale*min) - 128;
    q = round(scale*x + zeropoint), kept inside the int8 range.  The equation itself can
    exceed it by one: scale*max + zeropoint = 127 + frac(scale*min), and when that fraction
    is exactly one half the two roundings can put the maximum at 128; a code an int8 cache
    cannot hold is clipped to 127 (the paper stores int8 values, Sec. "Quantization")."""
    x = np.asarray(x, dtype=np.float64)
    lo, hi = float(x.min()), float(x.max())
    scale = 255.0 / (hi - lo)
    zeropoint = -np.rint(scale * lo) - 128.0
    q = np.clip(np.rint(scale * x + zeropoint), -128.0, 127.0)
    return q, scale, float(zeropoint)


def int8_dequantize(q: np.ndarray, scale: float, zeropoint: float) -> np.ndarray:
    """Eq. 4, last line: (q - zeropoint)/scale."""
    return (np.asarray(q, dtype=np.float64) - zeropoint) / scale


def int8_rows(z: np.ndarray) -> np.ndarray:
    """Latent rows as an int8 cache would return them (Sec. "Quantization", Eq. 4 applied on top of the
    autoencoder as in Table 5): every row is quantised with its own scale and zero-point - the paper does not
    state the granularity; a token's row is the unit that is written and read together - and dequantised again.
    A row of equal values has no range to scale and is kept as it is."""
    z = np.asarray(z, dtype=np.float64)
    out = np.empty_like(z)
    flat_in, flat_out = z.reshape(-1, z.shape[-1]), out.reshape(-1, z.shape[-1])
    for i, row in enumerate(flat_in):
        if row.max() == row.min():
            flat_out[i] = row
        else:
            q, scale, zp = int8_quantize(row)
            flat_out[i] = int8_dequantize(q, scale, zp)
    return out


# --------------------------------------------------------------------------
# Alg. 2, first steps: which heads may reuse the layer below
# --------------------------------------------------------------------------
def head_l1_distance(x: np.ndarray, n_kv_heads: int) -> np.ndarray:
    """Alg. 2, its distance step; Sec. "Network Architecture" describes the measure as the sum of
    absolute differences between two heads' key (value) matrices.  x: recorded K (or V) rows, [n_layers][n_rows][n_kv_heads *
    head_dim].  Returns D [n_layers - 1][n_kv_heads]: D[l-1][h] = mean over the rows and
    over head h's channels of |x[l] - x[l-1]|, i.e. the L1 norm of the difference of
    head h's matrix in layers l and l-1 divided by its element count (the paper does
    not say whether it normalises; dividing makes mini-batches of different sizes
    average as the text says they are averaged).  Same head index in both layers."""
    x = np.asarray(x, dtype=np.float64)
    n_layers, n_rows, width = x.shape
    hd = width // n_kv_heads
    out = np.zeros((n_layers - 1, n_kv_heads))
    for l in range(1, n_layers):
        diff = np.abs(x[l] - x[l - 1])
        for h in range(n_kv_heads):
            out[l - 1, h] = diff[:, h * hd:(h + 1) * hd].sum() / (n_rows * hd)
    return out


def reuse_map_from_l1(dist: np.ndarray, n_reuse: int) -> np.ndarray:
    """Alg. 2, next step: the heads with the smallest distance to the layer below
    reuse it (the paper picks its threshold empirically: here the threshold is given as
    a count, the n_reuse closest heads; equal distances go to the lower layer, then
    the lower head).  dist: [n_layers - 1][n_kv_heads] as returned above.  Returns the
    table in the form the cache takes it: int32 [n_layers * n_kv_heads], -1 = own
    data, else the head index in layer l-1 (always the same index here)."""
    dist = np.asarray(dist, dtype=np.float64)
    n_pairs, n_kv_heads = dist.shape
    order = sorted(range(n_pairs * n_kv_heads), key=lambda i: (dist[i // n_kv_heads, i % n_kv_heads], i))
    src = np.full((n_pairs + 1) * n_kv_heads, -1, dtype=np.int32)
    for i in order[:n_reuse]:
        src[n_kv_heads + i] = i % n_kv_heads
    return src


# --------------------------------------------------------------------------
# the autoencoder halves
# --------------------------------------------------------------------------
def mlp_forward(x: np.ndarray, w1, b1, bn, w2, b2, leaky_slope: float, bn_eps: float) -> np.ndarray:
    """FC -> BatchNorm(inference) -> LeakyReLU -> FC on rows of x.
    w1 [hidden, in], w2 [out, hidden] (row-major [out][in]); bn = [gamma, beta,
    running mean, running variance], each [hidden]."""
    x = np.asarray(x, dtype=np.float64)
    w1 = np.asarray(w1, np.float64); b1 = np.asarray(b1, np.float64)
    w2 = np.asarray(w2, np.float64); b2 = np.asarray(b2, np.float64)
    gamma, beta, mean, var = (np.asarray(r, np.float64) for r in bn)
    a = x @ w1.T + b1
    a = gamma * (a - mean) / np.sqrt(var + bn_eps) + beta
    a = np.where(a > 0, a, leaky_slope * a)
    return a @ w2.T + b2


def encode(ae: dict, x: np.ndarray) -> np.ndarray:
    return mlp_forward(x, ae["enc_w1"], ae["enc_b1"], ae["enc_bn"], ae["enc_w2"], ae["enc_b2"],
                       ae["leaky_slope"], ae["bn_eps"])


def decode(ae: dict, z: np.ndarray) -> np.ndarray:
    return mlp_forward(z, ae["dec_w1"], ae["dec_b1"], ae["dec_bn"], ae["dec_w2"], ae["dec_b2"],
                       ae["leaky_slope"], ae["bn_eps"])


# --------------------------------------------------------------------------
# the cache + attention
# --------------------------------------------------------------------------
class KVCAROracle:
    """Latent KV cache with cross-layer head reuse, and decode attention over it.

    storage: "exact" keeps latents in fp64; "f32"/"bf16" round each stored latent
    (the rounding is part of the cache format).  Every other intermediate is fp64.
    A (layer, which) without an autoencoder stores the raw rows of its stored heads.
    """

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 page_tokens: int, max_seqs: int, max_pages: int, storage: str = "exact"):
        assert n_q_heads % n_kv_heads == 0
        self.n_layers, self.hq, self.hkv, self.hd = n_layers, n_q_heads, n_kv_heads, head_dim
        self.P, self.max_seqs, self.max_pages = page_tokens, max_seqs, max_pages
        self.storage = storage
        self.src = [np.full((n_layers, n_kv_heads), -1, dtype=np.int64) for _ in (K, V)]
        self.ae: Dict[Tuple[int, int], dict] = {}
        # page bookkeeping: free pages are handed out in ascending order at first,
        # and a released page is the next one handed out (last in, first out)
        self.free_pages: List[int] = list(range(max_pages - 1, -1, -1))
        self.block_table: Dict[int, List[int]] = {}
        self.seq_len: Dict[int, int] = {}
        self.pool: Dict[Tuple[int, int], np.ndarray] = {}
        self.cur: Dict[Tuple[int, int, int], np.ndarray] = {}   # (layer, which, seq) -> exact row [W]

    # ---- reuse table ----------------------------------------------------
    def set_reuse_map(self, src_k: Sequence[int], src_v: Sequence[int]) -> None:
        for which, s in ((K, src_k), (V, src_v)):
            s = np.asarray(s, dtype=np.int64).reshape(self.n_layers, self.hkv)
            if np.any(s[0] != -1):
                raise ValueError("layer 0 has no layer below it")
            if np.any(s < -1) or np.any(s >= self.hkv):
                raise ValueError("head index out of range")
            self.src[which] = s.copy()

    def stored_heads(self, layer: int, which: int) -> List[int]:
        return [h for h in range(self.hkv) if self.src[which][layer, h] < 0]

    def resolve(self, layer: int, head: int, which: int) -> Tuple[int, int, int]:
        """Follow the table down until a head that keeps its own rows.
        Returns (root layer, root head, column slot of that head among the root
        layer's stored heads, in ascending head order)."""
        l, h = layer, head
        while self.src[which][l, h] >= 0:
            h = int(self.src[which][l, h])
            l -= 1
        slot = self.stored_heads(l, which).index(h)
        return l, h, slot

    # ---- autoencoders ---------------------------------------------------
    def set_autoencoder(self, layer: int, which: int, ae: dict) -> None:
        n = len(self.stored_heads(layer, which))
        if ae["in_dim"] != n * self.hd:
            raise ValueError("autoencoder must span exactly the stored heads")
        self.ae[(layer, which)] = ae

    def stored_width(self, layer: int, which: int) -> int:
        """Columns one cached token occupies in this layer's K or V pool."""
        n = len(self.stored_heads(layer, which))
        if (layer, which) in self.ae:
            return self.ae[(layer, which)]["latent"]
        return n * self.hd

    # ---- pages ----------------------------------------------------------
    def seq_open(self, seq: int) -> None:
        if seq in self.seq_len:
            raise ValueError("sequence already open")
        self.seq_len[seq] = 0
        self.block_table[seq] = []

    def seq_close(self, seq: int) -> None:
        for p in self.block_table.pop(seq):
            self.free_pages.append(p)
        del self.seq_len[seq]

    def reserve(self, seqs: Sequence[int], n_tokens: int) -> None:
        """Make sure pages exist for positions seq_len .. seq_len+n_tokens-1 of
        each sequence (in the order given); all or nothing."""
        need = []
        for s in seqs:
            have = len(self.block_table[s])
            want = (self.seq_len[s] + n_tokens + self.P - 1) // self.P
            need.append(max(0, want - have))
        if sum(need) > len(self.free_pages):
            raise MemoryError("out of pages")
        for s, n in zip(seqs, need):
            for _ in range(n):
                self.block_table[s].append(self.free_pages.pop())

    def locate(self, seq: int, token: int) -> Tuple[int, int]:
        """(physical page, pool row) of a logical token position."""
        page = self.block_table[seq][token // self.P]
        return page, page * self.P + token % self.P

    def _pool(self, layer: int, which: int) -> np.ndarray:
        key = (layer, which)
        if key not in self.pool:
            self.pool[key] = np.zeros((self.max_pages * self.P, self.stored_width(layer, which)))
        return self.pool[key]

    # ---- encode + append --------------------------------------------------
    def encode_append(self, layer: int, seqs: Sequence[int], n_tokens: int,
                      k: np.ndarray, v: np.ndarray) -> None:
        """k, v: [n_seqs, n_tokens, Hkv*hd] new rows.  The stored heads' slices
        are encoded (or kept raw) and written at positions seq_len.. of each
        sequence; the last token's exact rows are kept as the "current token"."""
        self.reserve(seqs, n_tokens)
        for which, x in ((K, k), (V, v)):
            x = np.asarray(x, dtype=np.float64).reshape(len(seqs), n_tokens, self.hkv * self.hd)
            heads = self.stored_heads(layer, which)
            for i, s in enumerate(seqs):
                self.cur[(layer, which, s)] = x[i, n_tokens - 1].copy()
            if not heads:
                continue
            cols = np.concatenate([np.arange(h * self.hd, (h + 1) * self.hd) for h in heads])
            pool = self._pool(layer, which)
            for i, s in enumerate(seqs):
                xs = x[i][:, cols]
                z = encode(self.ae[(layer, which)], xs) if (layer, which) in self.ae else xs
                z = round_to_storage(z, self.storage)
                for t in range(n_tokens):
                    _, row = self.locate(s, self.seq_len[s] + t)
                    pool[row] = z[t]

    def advance(self, seqs: Sequence[int], n_tokens: int) -> None:
        for s in seqs:
            self.seq_len[s] += n_tokens

    # ---- retrieve + restore -------------------------------------------------
    def restored_rows(self, layer: int, which: int, seq: int) -> np.ndarray:
        """All cached rows of `layer`'s own pool for one sequence, passed through
        that layer's decoder: [seq_len, n_stored*hd]."""
        L = self.seq_len[seq]
        pool = self._pool(layer, which)
        rows = [self.locate(seq, t)[1] for t in range(L)]
        z = pool[rows] if L else np.zeros((0, pool.shape[1]))
        if (layer, which) in self.ae:
            return decode(self.ae[(layer, which)], z)
        return z

    def head_rows(self, layer: int, head: int, which: int, seq: int, memo: Optional[dict] = None) -> np.ndarray:
        """Restored [seq_len, hd] rows that `head` of `layer` attends over."""
        rl, _, slot = self.resolve(layer, head, which)
        key = (rl, which, seq)
        if memo is not None and key in memo:
            full = memo[key]
        else:
            full = self.restored_rows(rl, which, seq)
            if memo is not None:
                memo[key] = full
        return full[:, slot * self.hd:(slot + 1) * self.hd]

    def current_row(self, layer: int, head: int, which: int, seq: int) -> np.ndarray:
        rl, rh, _ = self.resolve(layer, head, which)
        return self.cur[(rl, which, seq)][rh * self.hd:(rh + 1) * self.hd]

    # ---- attention --------------------------------------------------------
    def decode_attention(self, layer: int, seqs: Sequence[int], q: np.ndarray,
                         include_current: bool = True, return_probs: bool = False):
        """q: [n_seqs, Hq, hd].  Eq. 1 per query head over the restored cached
        rows of its KV head (query head i uses KV head i // (Hq/Hkv)) and, if
        include_current, the exact current-token K/V.  Returns [n_seqs, Hq, hd]."""
        q = np.asarray(q, dtype=np.float64).reshape(len(seqs), self.hq, self.hd)
        out = np.zeros_like(q)
        probs = []
        group = self.hq // self.hkv
        for i, s in enumerate(seqs):
            memo: dict = {}
            for qh in range(self.hq):
                g = qh // group
                keys = self.head_rows(layer, g, K, s, memo)
                vals = self.head_rows(layer, g, V, s, memo)
                if include_current:
                    keys = np.vstack([keys, self.current_row(layer, g, K, s)])
                    vals = np.vstack([vals, self.current_row(layer, g, V, s)])
                if keys.shape[0] == 0:
                    probs.append(np.zeros(0))
                    continue
                scores = keys @ q[i, qh] / math.sqrt(self.hd)
                e = np.exp(scores - scores.max())
                p = e / e.sum()
                out[i, qh] = p @ vals
                probs.append(p)
        return (out, probs) if return_probs else out

    # ---- accounting -------------------------------------------------------
    def cache_bytes_per_token(self) -> Tuple[float, float]:
        """(bytes one token occupies across all layers with the configured
        compression and reuse, bytes without either)."""
        b = STORAGE_BYTES[self.storage]
        comp = sum(self.stored_width(l, w) for l in range(self.n_layers) for w in (K, V)) * b
        if self.storage == "int8":   # per stored row: its scale and zero-point; the uncompressed reference is 16-bit
            comp += INT8_ROW_PARAM_BYTES * sum(1 for l in range(self.n_layers) for w in (K, V) if self.stored_width(l, w))
            b = 2
        full = 2 * self.n_layers * self.hkv * self.hd * b
        return float(comp), float(full)
