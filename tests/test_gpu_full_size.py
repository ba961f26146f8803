"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times
(whole batch, full cached length, every layer), on sampled outputs: the CUDA path runs
the whole workload, the CPU oracle mirrors a few sequences of it (all layers of those
sequences, so that reused heads find their root layers) and those sequences' outputs are
compared element by element.  Inputs come from torch's seeded device generator; the
sampled sequences' rows are copied to the host for the oracle."""
import numpy as np
import pytest
import torch

import kvcar_synth as synth
from kvcar_harness import Pair, assert_close
from paper_2512_06727_b200 import binding as B

pytestmark = pytest.mark.gpu


def _prefill_device(p, w, seqs, n_tokens, seed, chunk=1024):
    g = torch.Generator(device=p.s.device)
    g.manual_seed(seed)
    t = 0
    while t < n_tokens:
        n = min(chunk, n_tokens - t)
        for l in range(w.n_layers):
            k = torch.randn(len(seqs), n, w.kv_width, generator=g, device=p.s.device).to(p.s.dtype)
            v = torch.randn(len(seqs), n, w.kv_width, generator=g, device=p.s.device).to(p.s.dtype)
            p.append_device(l, seqs, k, v)
        torch.cuda.synchronize()
        p.advance(seqs, n)
        t += n
    p.s.ctx.sync_status(p.s.stream())


def _reused_heads(w):
    """(layer, head) pairs of the workload's seeded reuse map that read the layer below."""
    src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    return {(l, h) for l in range(w.n_layers) for h in range(w.n_kv_heads) if src[l * w.n_kv_heads + h] >= 0}


def _run(w, sampled, steps=1, fused=False, compress=True, absorbed=False):
    pps = (w.cached_tokens + steps + w.page_tokens - 1) // w.page_tokens
    p = Pair(w, max_seqs=w.batch, max_pages=w.batch * pps, max_pages_per_seq=pps, kernel=B.KERNEL_AUTO,
             compress=compress)
    p.oracle_seqs = set(sampled)
    seqs = list(range(w.batch))
    p.open(seqs)
    _prefill_device(p, w, seqs, w.cached_tokens, w.seed)
    want_kernel = B.KERNEL_TENSOR if compress else B.KERNEL_RAW
    assert all(p.s.ctx.layer_kernel(l) == want_kernel for l in range(w.n_layers))
    worst = 0.0
    pairs = set()
    for step in range(steps):
        res = p.decode_step(seqs, step, fused=fused, absorbed=absorbed)
        for l, (got, ref, rows) in res.items():
            assert rows == sorted(sampled)
            err, _ = assert_close(got[rows], ref, w.storage, f"{w.name} step {step} layer {l}")
            worst = max(worst, err)
            pairs |= {(s_, l) for s_ in sampled}
    comp, full = p.s.ctx.cache_bytes_per_token()
    assert (comp, full) == p.o.cache_bytes_per_token()
    # every output of a layer covers all of its KV heads, so a reused head is exercised iff its layer was compared
    hit = {(l, h) for (l, h) in _reused_heads(w) if any(pl == l for (_, pl) in pairs)}
    return worst, comp, full, pairs, hit


def test_config2_full_size_sampled():
    """GPT-2-small-shaped stack: 12 layers, batch 8, 1024 cached tokens, 25 % reuse; two steps;
    every sequence, i.e. every output of both steps (96 (sequence, layer) pairs per step), against the oracle."""
    w = synth.CONFIGS["c2"]
    worst, comp, full, pairs, hit = _run(w, list(range(w.batch)), steps=2)
    assert len(pairs) == 96 and hit == _reused_heads(w)
    assert comp < 0.5 * full      # latents halve the stored heads, reuse removes a quarter of them


def test_config3_full_size_sampled():
    """TinyLLaMA-shaped GQA stack: 22 layers, batch 32, 2048 cached tokens, 20 % reuse; two steps (the second reads
    the row the first appended); sequences 3, 17 and 30 against the oracle: 66 (sequence, layer) pairs, every layer
    and so every reused head."""
    w = synth.CONFIGS["c3"]
    _, _, _, pairs, hit = _run(w, [3, 17, 30], steps=2)
    assert len(pairs) == 66 and hit == _reused_heads(w)


def test_config4_long_context_sampled():
    """Long context: 32 768 cached tokens per sequence (256 tiles, split-KV over all of them), batch 4, all 22
    layers of the TinyLLaMA-shaped stack, two steps; sequences 0, 2 and 3 against the oracle: 66 (sequence, layer)
    pairs, every layer and every reused head of the seed-3 map."""
    w = synth.CONFIGS["c4"]
    _, _, _, pairs, hit = _run(w, [0, 2, 3], steps=2)
    assert len(pairs) == 66 and hit == _reused_heads(w)


def test_config5_batch_sweep_point_sampled():
    """GPT-2-small-shaped stack at 4096 cached tokens, batch 32 (one point of the batch sweep; many waves of
    clusters), all 12 layers, two steps; sequences 0, 5, 11, 17, 23 and 31 against the oracle: 72 (sequence, layer)
    pairs, every layer and every reused head of the seed-4 map."""
    w = synth.with_batch(synth.CONFIGS["c5"], 32)
    _, _, _, pairs, hit = _run(w, [0, 5, 11, 17, 23, 31], steps=2)
    assert len(pairs) == 72 and hit == _reused_heads(w)


@pytest.mark.parametrize("form", [True, "kv"], ids=["k", "k_and_v"])
def test_config5_absorbed_forms_sampled(form):
    """The same point of the batch sweep (GPT-2 shape, 4096 cached tokens, batch 32, all 12 layers with their reuse
    sources) through the absorbed last decoder layer - K side only, and both sides: two steps through the single-call
    step, sequences 0, 9, 16 and 31 against the oracle (48 (sequence, layer) pairs, every reused head)."""
    w = synth.with_batch(synth.CONFIGS["c5"], 32)
    _, _, _, pairs, hit = _run(w, [0, 9, 16, 31], steps=2, fused=True, absorbed=form)
    assert len(pairs) == 48 and hit == _reused_heads(w)


def test_config5_largest_batch_single_call_step_sampled():
    """The batch sweep's largest point: 256 sequences of 4096 cached tokens (8448 tiles, 57 tile pairs per
    cluster), all 12 layers, two steps, each layer's step through the single-call entry point; sequences 0, 63, 64,
    129, 200 and 255 against the oracle: 72 (sequence, layer) pairs, every layer and every reused head."""
    w = synth.with_batch(synth.CONFIGS["c5"], 256)
    _, _, _, pairs, hit = _run(w, [0, 63, 64, 129, 200, 255], steps=2, fused=True)
    assert len(pairs) == 72 and hit == _reused_heads(w)


def test_config3_uncompressed_twin_sampled():
    """Raw K/V pages at the TinyLLaMA shape, full batch and length, first six layers (reuse redirects heads to
    the lower layer's rows): the streaming kernel with 8 query heads per KV head."""
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=6)
    _run(w, [5, 31], steps=1, compress=False)


@pytest.mark.gpu
@pytest.mark.parametrize("cfg,batch", [("c5", 256), ("c3", 32)])
def test_fused_steps_back_to_back_equal_the_same_steps_synchronised(cfg, batch):
    """Three decode steps of the whole stack through kvcar_step_layer with nothing between the calls (the tile kernel
    of one layer on the side stream, the next layer's encoder behind it: how a serving loop and the bench drive the
    library), against the same three steps on a second, identically filled context with a device synchronise after
    every layer: no device error, guard regions intact, outputs bit-equal.  The element-wise parity tests synchronise
    per layer (they copy every output back), so only this test sees the launches overlap at full size."""
    import bench
    w = synth.scaled(synth.CONFIGS[cfg], batch=batch)

    class A:
        pass
    outs = []
    for synchronise in (False, True):
        a2 = A()
        a2.uncompressed = False
        a2.kernel = "auto"
        sess, src, aes = bench.build_session(w, a2, torch, 3 + 24)
        sess.has_autoencoders = bool(aes)
        bench.fast_prefill(sess, w, torch)
        seqs = list(range(w.batch))
        stream = sess.stream()
        k, v, q, out = bench.step_inputs(sess, w, torch, 3)
        for i in range(3):
            for l in range(w.n_layers):
                sess.ctx.step_layer(l, seqs, k[i, l].data_ptr(), v[i, l].data_ptr(), q[i, l].data_ptr(),
                                    out[i, l].data_ptr(), B.INCLUDE_CURRENT_EXACT, stream)
                if synchronise:
                    torch.cuda.synchronize()
            sess.ctx.advance(seqs, 1, stream)
        torch.cuda.synchronize()
        sess.ctx.sync_status(stream)
        assert sess.ctx.debug_check(stream) == (0, 0, -1)
        assert bool(torch.isfinite(out.float()).all())
        outs.append(out.clone())
        del sess
    assert torch.equal(outs[0], outs[1])
