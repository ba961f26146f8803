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


def _run(w, sampled, steps=1, fused=False, compress=True):
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
    for step in range(steps):
        res = p.decode_step(seqs, step, fused=fused)
        for l, (got, ref, rows) in res.items():
            assert rows == sorted(sampled)
            err, _ = assert_close(got[rows], ref, w.storage, f"{w.name} step {step} layer {l}")
            worst = max(worst, err)
    comp, full = p.s.ctx.cache_bytes_per_token()
    assert (comp, full) == p.o.cache_bytes_per_token()
    return worst, comp, full


def test_config2_full_size_sampled():
    """GPT-2-small-shaped stack: 12 layers, batch 8, 1024 cached tokens, 25 % reuse; two steps;
    every sequence, i.e. every output of both steps, against the oracle."""
    w = synth.CONFIGS["c2"]
    worst, comp, full = _run(w, list(range(w.batch)), steps=2)
    assert comp < 0.5 * full      # latents halve the stored heads, reuse removes a quarter of them


def test_config3_full_size_sampled():
    """TinyLLaMA-shaped GQA stack: 22 layers, batch 32, 2048 cached tokens, 20 % reuse;
    sequences 3, 17 and 30 against the oracle: 66 (sequence, layer) pairs, every layer and so every reused head."""
    w = synth.CONFIGS["c3"]
    _run(w, [3, 17, 30], steps=1)


def test_config4_long_context_sampled():
    """Long context: 32 768 cached tokens per sequence (256 tiles, split-KV over all of them),
    batch 4, the first three layers of the TinyLLaMA-shaped stack (the oracle would need
    hours for all 22 at this length); sequence 2 against the oracle."""
    w = synth.scaled(synth.CONFIGS["c4"], n_layers=3)
    _run(w, [2], steps=1)


def test_config5_batch_sweep_point_sampled():
    """GPT-2-small-shaped stack at 4096 cached tokens, batch 32 (one point of the batch
    sweep; many waves of clusters), first four layers; sequence 17 against the oracle."""
    w = synth.scaled(synth.with_batch(synth.CONFIGS["c5"], 32), n_layers=4)
    _run(w, [17], steps=1)


def test_config5_largest_batch_single_call_step_sampled():
    """The batch sweep's largest point: 256 sequences of 4096 cached tokens (8448 tiles, 57 tile pairs per
    cluster), first two layers, each layer's step through the single-call entry point; the first and the last
    sequence against the oracle."""
    w = synth.scaled(synth.with_batch(synth.CONFIGS["c5"], 256), n_layers=2)
    _run(w, [0, 255], steps=1, fused=True)


def test_config3_uncompressed_twin_sampled():
    """Raw K/V pages at the TinyLLaMA shape, full batch and length, first six layers (reuse redirects heads to
    the lower layer's rows): the streaming kernel with 8 query heads per KV head."""
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=6)
    _run(w, [5, 31], steps=1, compress=False)
