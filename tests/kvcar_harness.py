"""Drives the CPU oracle and the CUDA library side by side on the same seeded
inputs.  The two never see each other: inputs come from kvcar_synth (or, for
full-size runs, from torch's seeded device generator and are copied back to the
host for the oracle), outputs are compared here."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

import kvcar_synth as synth
from oracle.kvcar_oracle import K, V, KVCAROracle
from paper_2512_06727_b200 import binding as B
from paper_2512_06727_b200.session import Session

# tolerances of the decode output (max abs; relative L2) per storage type
TOL = {"f32": (1e-4, 1e-4), "bf16": (2e-2, 1e-2)}


def latent_tol(storage: str, z_ref: np.ndarray, bf16_hidden: bool = False) -> np.ndarray:
    """Stored latents: one storage ulp (rare rounding ties after fp32 accumulation) plus fp32 noise.
    bf16_hidden (the tensor-core encoder): each of the m terms w2[i][j] * a[j] of a latent also carries the bf16
    rounding of a[j] (relative <= 2^-9); with terms of either sign a latent moves by about 2^-9 / sqrt(3) of the
    row's scale, so 2^-7 of the row's RMS latent (about seven standard deviations) is allowed on top."""
    if storage == "bf16":
        tol = 2.0 ** -7 * np.abs(z_ref) + 1e-6
        if bf16_hidden:
            tol = tol + 2.0 ** -7 * np.sqrt(np.mean(np.square(z_ref), axis=-1, keepdims=True))
        return tol
    return 1e-5 * (1.0 + np.abs(z_ref))


class Pair:
    def __init__(self, w: synth.Workload, max_seqs: int, max_pages: int, max_pages_per_seq: int,
                 src_k: Optional[np.ndarray] = None, src_v: Optional[np.ndarray] = None,
                 compressed_layers: Optional[List[int]] = None, compress: bool = True,
                 kernel: int = B.KERNEL_AUTO, with_oracle: bool = True, ae_kwargs: Optional[dict] = None,
                 latent_quant: bool = False):
        """latent_quant: int8 latent rows (Eq. 4) on both sides; inputs and weights stay on w.storage's grid."""
        self.w = w
        self.latent_quant = latent_quant
        n = w.n_layers * w.n_kv_heads
        if src_k is None:
            src_k = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
        if src_v is None:
            src_v = src_k.copy()
        self.src_k, self.src_v = src_k, src_v
        self.aes = synth.make_stack_autoencoders(w, src_k, src_v, layers=compressed_layers,
                                                 **(ae_kwargs or {})) if compress else {}
        self.o = None
        if with_oracle:
            self.o = KVCAROracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, max_seqs,
                                 max_pages, "int8" if latent_quant else w.storage)
            self.o.set_reuse_map(src_k, src_v)
            for (l, which), ae in self.aes.items():
                self.o.set_autoencoder(l, which, ae)
        self.s = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, max_seqs, max_pages,
                         max_pages_per_seq, w.storage, src_k, src_v, self.aes, kernel=kernel,
                         latent_quant=latent_quant)
        self.oracle_seqs: Optional[set] = None     # None = the oracle mirrors every sequence

    # ------------------------------------------------------------------
    def open(self, seqs: Sequence[int]):
        for s in seqs:
            self.s.ctx.seq_open(s)
            if self.o is not None and (self.oracle_seqs is None or s in self.oracle_seqs):
                self.o.seq_open(s)

    def _oracle_rows(self, seqs):
        return [i for i, s in enumerate(seqs) if self.oracle_seqs is None or s in self.oracle_seqs]

    def append(self, layer: int, seqs: Sequence[int], k: np.ndarray, v: np.ndarray, tensor: bool = False):
        """k, v: host float arrays [n_seqs, n_tokens, W] already on the storage grid.  tensor: through the
        tensor-core bulk encoder instead of kvcar_encode_append."""
        n_tokens = k.shape[1]
        dk, dv = self.s.to_device(k), self.s.to_device(v)
        call = self.s.ctx.encode_append_tensor if tensor else self.s.ctx.encode_append
        call(layer, list(seqs), n_tokens, dk.data_ptr(), dv.data_ptr(), self.s.stream())
        torch.cuda.current_stream().synchronize()
        if self.o is not None:
            rows = self._oracle_rows(seqs)
            if rows:
                self.o.encode_append(layer, [seqs[i] for i in rows], n_tokens, k[rows], v[rows])

    def append_device(self, layer: int, seqs: Sequence[int], dk: torch.Tensor, dv: torch.Tensor):
        """Same with inputs already on the device (full-size runs)."""
        n_tokens = dk.shape[1]
        self.s.ctx.encode_append(layer, list(seqs), n_tokens, dk.data_ptr(), dv.data_ptr(), self.s.stream())
        if self.o is not None:
            rows = self._oracle_rows(seqs)
            if rows:
                idx = torch.tensor(rows, device=dk.device)
                hk = dk.index_select(0, idx).float().cpu().numpy()
                hv = dv.index_select(0, idx).float().cpu().numpy()
                self.o.encode_append(layer, [seqs[i] for i in rows], n_tokens, hk, hv)

    def advance(self, seqs: Sequence[int], n: int):
        self.s.ctx.advance(list(seqs), n, self.s.stream())
        if self.o is not None:
            rows = self._oracle_rows(seqs)
            if rows:
                self.o.advance([seqs[i] for i in rows], n)

    def prefill(self, seqs: Sequence[int], n_tokens: int, t0: int = 0, tensor: bool = False):
        w = self.w
        for l in range(w.n_layers):
            k = np.stack([synth.make_kv(w, l, K, s, t0, n_tokens) for s in seqs])
            v = np.stack([synth.make_kv(w, l, V, s, t0, n_tokens) for s in seqs])
            self.append(l, seqs, k, v, tensor=tensor)
        self.advance(seqs, n_tokens)

    def attention(self, layer: int, seqs: Sequence[int], q: np.ndarray, include_current: bool = True,
                  absorbed: bool = False):
        """Returns (gpu [n,Hq,hd] float64, oracle rows or None, row indices the oracle covers)."""
        dq = self.s.to_device(q)
        out = torch.empty_like(dq)
        flags = (B.INCLUDE_CURRENT_EXACT if include_current else 0) | \
                (B.ABSORBED if absorbed else 0) | (B.ABSORBED_V if absorbed == "kv" else 0)
        self.s.ctx.decode_attention(layer, list(seqs), dq.data_ptr(), out.data_ptr(), flags, self.s.stream())
        self.s.ctx.sync_status(self.s.stream())
        got = out.float().cpu().numpy().astype(np.float64)
        ref, rows = None, []
        if self.o is not None:
            rows = self._oracle_rows(seqs)
            if rows:
                ref = self.o.decode_attention(layer, [seqs[i] for i in rows], q[rows], include_current=include_current)
        return got, ref, rows

    def step_layer(self, layer: int, seqs: Sequence[int], k: np.ndarray, v: np.ndarray, q: np.ndarray,
                   include_current: bool = True, absorbed: bool = False):
        """append + attention of one layer through the single-call entry point; same return as attention()."""
        dk, dv, dq = self.s.to_device(k), self.s.to_device(v), self.s.to_device(q)
        out = torch.empty_like(dq)
        flags = (B.INCLUDE_CURRENT_EXACT if include_current else 0) | \
                (B.ABSORBED if absorbed else 0) | (B.ABSORBED_V if absorbed == "kv" else 0)
        self.s.ctx.step_layer(layer, list(seqs), dk.data_ptr(), dv.data_ptr(), dq.data_ptr(), out.data_ptr(), flags,
                              self.s.stream())
        self.s.ctx.sync_status(self.s.stream())
        got = out.float().cpu().numpy().astype(np.float64)
        ref, rows = None, []
        if self.o is not None:
            rows = self._oracle_rows(seqs)
            if rows:
                sub = [seqs[i] for i in rows]
                self.o.encode_append(layer, sub, 1, k[rows], v[rows])
                ref = self.o.decode_attention(layer, sub, q[rows], include_current=include_current)
        return got, ref, rows

    def decode_step(self, seqs: Sequence[int], step: int, q_scale: float = 1.0, include_current: bool = True,
                    layers: Optional[Sequence[int]] = None, fused: bool = False, absorbed: bool = False):
        """One full decode step (encode-append + attention for every layer, then
        advance).  Returns per-layer (gpu, oracle, rows).  fused: each layer through
        the single-call entry point instead of the two calls."""
        w = self.w
        res = {}
        t = {s: self.s.ctx.seq_len(s) for s in seqs}
        for l in range(w.n_layers):
            k = np.stack([synth.make_kv(w, l, K, s, t[s], 1) for s in seqs])
            v = np.stack([synth.make_kv(w, l, V, s, t[s], 1) for s in seqs])
            if fused:
                q = np.stack([synth.make_q(w, l, s, step, scale=q_scale) for s in seqs])
                res[l] = self.step_layer(l, seqs, k, v, q, include_current, absorbed)
                continue
            self.append(l, seqs, k, v)
            if layers is None or l in layers:
                q = np.stack([synth.make_q(w, l, s, step, scale=q_scale) for s in seqs])
                res[l] = self.attention(l, seqs, q, include_current, absorbed)
        self.advance(seqs, 1)
        return res

    # ------------------------------------------------------------------
    def check_latents(self, seqs: Sequence[int], bf16_hidden: bool = False):
        """Every cached row of every layer against the oracle's, plus exact page/row indices."""
        w = self.w
        worst = 0.0
        for s in seqs:
            L = self.o.seq_len[s]
            assert self.s.ctx.seq_len(s) == L
            rows = []
            for t in range(L):
                assert self.s.ctx.debug_locate(s, t) == self.o.locate(s, t)
                rows.append(self.o.locate(s, t)[1])
            if not rows:
                continue
            for l in range(w.n_layers):
                for which in (K, V):
                    if self.o.stored_width(l, which) == 0:
                        continue
                    ref = self.o._pool(l, which)[rows]
                    if self.latent_quant:
                        worst = max(worst, self._check_int8_rows(l, which, rows, ref))
                        continue
                    got = self.s.pool_rows(l, which)[torch.tensor(rows, device=self.s.device)].float().cpu().numpy()
                    err = np.abs(got - ref)
                    tol = latent_tol(w.storage, ref, bf16_hidden)
                    assert np.all(err <= tol), (l, which, s, float((err - tol).max()))
                    worst = max(worst, float(err.max()))
        return worst


    def _check_int8_rows(self, l: int, which: int, rows, ref: np.ndarray) -> float:
        """int8 rows: the oracle keeps each row as Eq. 4 returns it, x' = (q - zp)/scale with scale = 255/(max-min).
        The library's latents carry fp32 rounding, so its row range, scale and zero-point differ by a few fp32 ulps
        and a code may fall on the other side of a rounding boundary: a restored value may be off by one code step
        (1/scale = range/255) plus the fp32 noise, never more.  The codes are int8 and the parameters finite."""
        idx = torch.tensor(rows, device=self.s.device)
        q = self.s.pool_rows(l, which)[idx]
        assert q.dtype == torch.int8
        par = self.s.pool_quant_params(l, which)[idx].cpu().numpy().astype(np.float64)
        scale, zp = par[:, :1], par[:, 1:]
        assert np.all(np.isfinite(par)) and np.all(scale > 0)
        assert np.all(zp == np.rint(zp)), "zero-points are whole numbers (Eq. 4)"
        got = (q.cpu().numpy().astype(np.float64) - zp) / scale
        rng = ref.max(axis=1, keepdims=True) - ref.min(axis=1, keepdims=True)
        # the oracle's row spans exactly 255 code steps
        np.testing.assert_allclose(scale * rng, 255.0, rtol=1e-4)
        err = np.abs(got - ref)
        tol = 1.02 * rng / 255.0 + 1e-5
        assert np.all(err <= tol), (l, which, float((err / tol).max()))
        # and almost every code agrees: a step of difference only at a rounding boundary
        assert np.mean(err > 0.02 * rng / 255.0 + 1e-5) < 0.02, (l, which, float(np.mean(err > 0.02 * rng / 255.0)))
        return float(err.max())


def assert_close(got: np.ndarray, ref: np.ndarray, storage: str, what=""):
    max_abs, rel_l2 = TOL[storage]
    err = float(np.max(np.abs(got - ref))) if got.size else 0.0
    denom = float(np.linalg.norm(ref))
    rel = float(np.linalg.norm(got - ref)) / denom if denom > 0 else 0.0
    assert err <= max_abs, f"{what}: max abs error {err:.3e} > {max_abs}"
    assert rel <= rel_l2, f"{what}: relative L2 error {rel:.3e} > {rel_l2}"
    return err, rel
