"""The tensor-core bulk encoder (kvcar_encode_append_tensor) against the CPU oracle: the cache rows it writes,
and decode attention over a cache it filled."""
import numpy as np
import pytest
import torch

import kvcar_synth as synth
from kvcar_harness import Pair, assert_close
from paper_2512_06727_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", ["c2", "c3"])
def test_tensor_prefill_rows_and_decode_over_them(cfg):
    """A stack with reuse (so encoder widths differ by layer and between K and V), sequences whose rows end
    inside a 128-row tile, a second bulk append on top of the first (rows land behind existing ones, across a page
    boundary), then a decode step through the ordinary path over the cache the tensor-core encoder wrote."""
    w = synth.scaled(synth.CONFIGS[cfg], n_layers=4, batch=3, cached_tokens=0, decode_steps=1, reuse_frac=0.3)
    src_k = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    src_v = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed + 3)
    p = Pair(w, max_seqs=3, max_pages=36, max_pages_per_seq=12, src_k=src_k, src_v=src_v)
    seqs = [0, 1, 2]
    p.open(seqs)
    p.prefill(seqs, 200, tensor=True)              # 600 rows: four full row tiles and one of 88 rows
    p.prefill([1], 77, t0=200, tensor=True)        # behind existing rows, ends inside a page
    p.prefill([0, 2], 1, t0=200, tensor=True)      # a single token per sequence also goes through
    p.check_latents(seqs, bf16_hidden=True)
    res = p.decode_step(seqs, 0)
    for l, (got, ref, rows) in res.items():
        assert_close(got[rows], ref, "bf16", f"{cfg} layer {l} over tensor-prefilled cache")


def test_tensor_prefill_matches_the_fp32_hidden_encoder_closely():
    """The same rows through both encoders: the two caches agree within the bf16-hidden tolerance, row for row."""
    w = synth.scaled(synth.CONFIGS["c2"], n_layers=2, batch=2, cached_tokens=0, decode_steps=1, reuse_frac=0.0)
    caches = []
    for tensor in (False, True):
        p = Pair(w, max_seqs=2, max_pages=8, max_pages_per_seq=4, with_oracle=False)
        p.open([0, 1])
        p.prefill([0, 1], 130, tensor=tensor)
        caches.append([p.s.pool_rows(l, which).float().cpu().numpy() for l in range(w.n_layers) for which in (0, 1)])
    for a, b in zip(*caches):
        used = np.abs(a).sum(axis=-1) > 0            # rows that were written
        assert used.sum() == 260
        scale = np.sqrt(np.mean(np.square(a[used]), axis=-1, keepdims=True))
        assert np.all(np.abs(a[used] - b[used]) <= 2.0 ** -7 * np.abs(a[used]) + 2.0 ** -7 * scale + 1e-6)


def test_tensor_prefill_refuses_what_it_cannot_do():
    w = synth.scaled(synth.CONFIGS["c2"], n_layers=1, batch=1, reuse_frac=0.0)
    p = Pair(w, max_seqs=1, max_pages=4, max_pages_per_seq=4, compress=False, with_oracle=False)   # raw layers
    p.open([0])
    k = torch.zeros(1, 4, w.kv_width, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.KvcarError) as e:
        p.s.ctx.encode_append_tensor(0, [0], 4, k.data_ptr(), k.data_ptr(), p.s.stream())
    assert e.value.status == 5          # KVCAR_ERR_UNSUPPORTED
    assert p.s.ctx.seq_len(0) == 0
