"""kvcar_decode_attention_static: the decode-attention call for callers that
cannot allocate device memory (a server whose arena already owns the whole
device budget, a plugin handed tensors but no allocator, a decode loop where a
driver allocation would stall the GPU).  Its split-KV scratch is a fixed array
inside the library, so the test checks that, through the C ABI, it returns what
the regular entry point returns, twice in a row (the second call reuses the
array with the first call's leftovers in it), and that a request larger than the
array is refused before anything is launched.

This file sorts last on purpose: a run that stops at the first failure has then
already executed every other test."""
import numpy as np
import pytest
import torch

import kvcar_synth as synth
from kvcar_harness import TOL, Pair
from oracle.kvcar_oracle import K, V
from paper_2512_06727_b200 import binding as B

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_regular_one_twice():
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=3, batch=3, reuse_frac=0.34)
    p = Pair(w, max_seqs=3, max_pages=16, max_pages_per_seq=6, kernel=B.KERNEL_GENERIC)
    seqs = [0, 1, 2]
    p.open(seqs)
    p.prefill([0], 300)       # three chunks
    p.prefill([1], 129)       # two chunks, ragged
    p.prefill([2], 5)
    max_abs, rel_l2 = TOL["bf16"]
    for call in range(2):     # second call: shorter list, other layer, other queries -> stale scratch contents
        layer = 2 - call
        use = seqs if call == 0 else [1, 2]
        for l in range(w.n_layers):
            k = np.stack([synth.make_kv(w, l, K, s, 400 + call, 1) for s in use])
            v = np.stack([synth.make_kv(w, l, V, s, 400 + call, 1) for s in use])
            p.append(l, use, k, v)
        qh = np.stack([synth.make_q(w, layer, s, call) for s in use])
        q = p.s.to_device(qh)
        ref = torch.empty_like(q)
        got = torch.full_like(q, float("nan"))
        p.s.ctx.decode_attention(layer, use, q.data_ptr(), ref.data_ptr(), B.INCLUDE_CURRENT_EXACT, p.s.stream())
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        p.s.ctx.decode_attention_static(layer, use, q.data_ptr(), got.data_ptr(), B.INCLUDE_CURRENT_EXACT,
                                        p.s.stream())
        p.s.ctx.sync_status(p.s.stream())
        # the array was set aside when memory was bound: the call itself leaves the device's free memory as it was
        assert torch.cuda.mem_get_info()[0] == free_before
        a, b = got.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.all(np.isfinite(a))
        # same kernels, same order of operations, only the scratch lives elsewhere: the same bits
        assert np.array_equal(a, b)
        # and both are the method's result: against the oracle, at the tolerance of every other parity test
        want = p.o.decode_attention(layer, use, qh)
        assert np.max(np.abs(a - want)) <= max_abs
        assert np.linalg.norm(a - want) <= rel_l2 * np.linalg.norm(want)


def test_static_scratch_rejects_oversized_requests():
    # 4 sequences x 256 chunks x 32 heads x 66 floats = 8.25 MiB of partials > the 8 MiB array
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=1, batch=4, reuse_frac=0.0)
    p = Pair(w, max_seqs=4, max_pages=4 * 512, max_pages_per_seq=512, kernel=B.KERNEL_GENERIC, with_oracle=False)
    seqs = [0, 1, 2, 3]
    p.open(seqs)
    p.s.ctx.reserve(seqs, 32768)
    p.s.ctx.advance(seqs, 32768, p.s.stream())
    q = torch.zeros(4, w.n_q_heads, w.head_dim, dtype=p.s.dtype, device="cuda")
    launches = p.s.ctx.launch_count()
    with pytest.raises(B.KvcarError) as e:
        p.s.ctx.decode_attention_static(0, seqs, q.data_ptr(), q.data_ptr(), 0, p.s.stream())
    assert e.value.status == 4 and "static scratch too small" in str(e.value)
    assert p.s.ctx.launch_count() == launches
    p.s.ctx.sync_status(p.s.stream())
