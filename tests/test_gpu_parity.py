"""GPU parity: the CUDA library against the CPU oracle, element by element, on
the same seeded inputs, through the C ABI.  Sizes are chosen so that the oracle
finishes in seconds while the kernels still see several tiles, several pages and
ragged tails."""
import numpy as np
import pytest
import torch

import kvcar_synth as synth
from kvcar_harness import Pair, assert_close
from oracle.kvcar_oracle import K, V
from paper_2512_06727_b200 import binding as B

pytestmark = pytest.mark.gpu

KERNELS = [B.KERNEL_GENERIC, B.KERNEL_AUTO]
KNAME = {B.KERNEL_GENERIC: "generic", B.KERNEL_AUTO: "auto"}


def _check_step(res, storage, what):
    worst = 0.0
    for l, (got, ref, rows) in res.items():
        err, rel = assert_close(got[rows], ref, storage, f"{what} layer {l}")
        worst = max(worst, err)
    return worst


def test_config1_fp32_single_layer():
    """Configuration 1 exactly: one GPT-2-small-shaped layer, 768->384, batch 1,
    128 cached tokens, one decode step, fp32, no reuse; max abs error <= 1e-4."""
    w = synth.CONFIGS["c1"]
    p = Pair(w, max_seqs=1, max_pages=4, max_pages_per_seq=4)
    p.open([0])
    p.prefill([0], w.cached_tokens)
    p.check_latents([0])
    res = p.decode_step([0], 0)
    got, ref, rows = res[0]
    err, rel = assert_close(got[rows], ref, "f32", "config 1")
    assert err <= 1e-4
    assert p.s.ctx.cache_bytes_per_token() == (2 * 384 * 4, 2 * 768 * 4)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_gpt2_shape_stack_bf16_with_reuse(kernel):
    """Config-2-shaped stack (12 layers x 12 heads, latent 32/head, 25 % reuse),
    reduced batch and ragged lengths, two decode steps with encode-append."""
    w = synth.scaled(synth.CONFIGS["c2"], batch=3, cached_tokens=0, decode_steps=2)
    p = Pair(w, max_seqs=4, max_pages=16, max_pages_per_seq=5, kernel=kernel)
    seqs = [2, 0, 3]
    p.open(seqs)
    p.prefill([2], 200)
    p.prefill([0], 131)
    p.prefill([3], 64)
    p.check_latents(seqs)
    if kernel == B.KERNEL_AUTO:     # the bf16 stack must really run on the tensor-core kernel
        assert all(p.s.ctx.layer_kernel(l) == B.KERNEL_TENSOR for l in range(w.n_layers))
    for step in range(2):
        _check_step(p.decode_step(seqs, step), "bf16", f"step {step}")
    p.check_latents(seqs)
    assert p.s.ctx.cache_bytes_per_token() == p.o.cache_bytes_per_token()


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_tinyllama_shape_gqa_stack_bf16_with_reuse(kernel):
    """Config-3-shaped GQA stack (22 layers, 32 query / 4 KV heads, latent 32/head,
    20 % reuse), K and V reuse maps different, ragged lengths incl. 1 token."""
    w = synth.scaled(synth.CONFIGS["c3"], batch=4, cached_tokens=0, decode_steps=2)
    src_k = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    src_v = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed + 7)
    p = Pair(w, max_seqs=4, max_pages=20, max_pages_per_seq=6, src_k=src_k, src_v=src_v, kernel=kernel)
    seqs = [0, 1, 2, 3]
    p.open(seqs)
    for s, n in zip(seqs, (300, 257, 128, 1)):
        p.prefill([s], n)
    p.check_latents(seqs)
    if kernel == B.KERNEL_AUTO:
        assert all(p.s.ctx.layer_kernel(l) == B.KERNEL_TENSOR for l in range(w.n_layers))
    for step in range(2):
        _check_step(p.decode_step(seqs, step), "bf16", f"step {step}")


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_peaked_softmax_and_planted_key(kernel):
    """N(0,1) inputs give near-uniform softmax, under which a token-indexing bug
    hardly moves the output: repeat with queries scaled x8 and with one cached key
    made proportional to the query."""
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=3, batch=2, cached_tokens=0, decode_steps=1, reuse_frac=0.34)
    p = Pair(w, max_seqs=2, max_pages=12, max_pages_per_seq=6, kernel=kernel)
    seqs = [0, 1]
    p.open(seqs)
    p.prefill(seqs, 333)
    res = p.decode_step(seqs, 0, q_scale=8.0)
    _check_step(res, "bf16", "q x8")
    # the softmax really is peaked: the largest probability of some head exceeds 0.5
    out, probs = p.o.decode_attention(2, [0], np.stack([synth.make_q(w, 2, 0, 0, scale=8.0)]),
                                      include_current=False, return_probs=True)
    assert max(float(pr.max()) for pr in probs) > 0.5
    # planted key: make token 77's pre-compression K of every head a multiple of one query head, raw layer 0
    w2 = synth.scaled(w, n_layers=1, reuse_frac=0.0)
    p2 = Pair(w2, max_seqs=1, max_pages=4, max_pages_per_seq=4, compress=False, kernel=kernel)
    p2.open([0])
    q = synth.make_q(w2, 0, 0, 0)
    k = synth.make_kv(w2, 0, K, 0, 0, 150)[None].copy()
    v = synth.make_kv(w2, 0, V, 0, 0, 150)[None].copy()
    for g in range(w2.n_kv_heads):
        k[0, 77, g * 64:(g + 1) * 64] = synth.to_bf16_grid(6.0 * q[g * 8])
    p2.append(0, [0], k, v)
    p2.advance([0], 150)
    got, ref, rows = p2.attention(0, [0], q[None], include_current=False)
    assert_close(got, ref, "bf16", "planted key")
    for g in range(w2.n_kv_heads):   # head g*8 attends almost only to token 77
        assert np.max(np.abs(got[0, g * 8] - v[0, 77, g * 64:(g + 1) * 64])) < 0.05


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_edge_cases_empty_current_only_and_single_token(kernel):
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, batch=3, reuse_frac=0.5)
    p = Pair(w, max_seqs=3, max_pages=8, max_pages_per_seq=3, kernel=kernel)
    seqs = [0, 1, 2]
    p.open(seqs)
    p.prefill([1], 1)
    p.prefill([2], 65)
    # seq 0 has nothing cached: with the current token the output is that token's exact V
    res = p.decode_step(seqs, 0)
    _check_step(res, "bf16", "current only")
    # nothing cached and no current token: zeros
    p3 = Pair(w, max_seqs=1, max_pages=2, max_pages_per_seq=2, kernel=kernel)
    p3.open([0])
    got, ref, rows = p3.attention(0, [0], synth.make_q(w, 0, 0, 0)[None], include_current=False)
    assert np.all(got == 0) and np.all(ref == 0)
    # cached tokens only (current token attended through its latent after advance)
    got, ref, rows = p.attention(1, seqs, np.stack([synth.make_q(w, 1, s, 9) for s in seqs]), include_current=False)
    assert_close(got, ref, "bf16", "cached only")


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_uncompressed_twin_and_mixed_stack(kernel):
    """No autoencoders (raw K/V pages, reuse still redirects heads) and a stack
    with autoencoders in some layers only (Table 2's "N layers" rows)."""
    w = synth.scaled(synth.CONFIGS["c2"], n_layers=4, batch=2, reuse_frac=0.3)
    for layers, compress in ((None, False), ([1, 2], True)):
        p = Pair(w, max_seqs=2, max_pages=8, max_pages_per_seq=4, compressed_layers=layers, compress=compress,
                 kernel=kernel)
        p.open([0, 1])
        p.prefill([0], 190)
        p.prefill([1], 70)
        p.check_latents([0, 1])
        _check_step(p.decode_step([0, 1], 0), "bf16", f"layers={layers}")
        assert p.s.ctx.cache_bytes_per_token() == p.o.cache_bytes_per_token()


@pytest.mark.parametrize("heads", [(32, 4), (12, 4), (6, 2)], ids=["group8", "group3", "group3_two_kv_heads"])
def test_uncompressed_twin_with_query_groups(heads):
    """Raw K/V pages with several query heads per KV head: the streaming kernel runs the group's dots on the
    warp-level tensor op (groups of more than two heads).  Ragged tiles: a 32-token step that ends inside a tile,
    a tile of one token, page boundaries inside a step; reuse redirects heads to the lower layer's rows."""
    hq, hkv = heads
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=3, n_q_heads=hq, n_kv_heads=hkv, batch=4, reuse_frac=0.4)
    p = Pair(w, max_seqs=4, max_pages=24, max_pages_per_seq=8, compress=False)
    seqs = [0, 1, 2, 3]
    p.open(seqs)
    for s_, n in zip(seqs, (300, 129, 33, 1)):
        p.prefill([s_], n)
    assert all(p.s.ctx.layer_kernel(l) == B.KERNEL_RAW for l in range(w.n_layers))
    for step in range(2):
        _check_step(p.decode_step(seqs, step), "bf16", f"raw group {hq // hkv} step {step}")


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_physical_page_permutation_is_bit_invariant(kernel):
    """The same logical cache laid out on different physical pages must give
    bit-identical outputs."""
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, batch=1, reuse_frac=0.25)

    def run(scramble):
        p = Pair(w, max_seqs=3, max_pages=12, max_pages_per_seq=6, kernel=kernel, with_oracle=False)
        if scramble:
            p.open([1, 2])
            p.s.ctx.reserve([1], 130); p.s.ctx.reserve([2], 70)
            p.s.ctx.seq_close(1); p.s.ctx.seq_close(2)
        p.open([0])
        p.prefill([0], 200)
        pages = [p.s.ctx.debug_locate(0, t)[0] for t in range(0, 200, 64)]
        res = p.decode_step([0], 0)
        return pages, {l: r[0] for l, r in res.items()}
    pa, a = run(False)
    pb, b = run(True)
    assert pa != pb
    for l in a:
        assert np.array_equal(a[l], b[l])


def test_large_grid_runs_k_then_v_in_one_cluster():
    """More tile pairs than a quarter of the SMs: the tensor-core kernel stops spreading a
    pair over several clusters and each cluster restores K, then V (the other tests are
    small enough to take the split paths)."""
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, batch=5, cached_tokens=0, decode_steps=1, reuse_frac=0.25)
    pps = 34
    p = Pair(w, max_seqs=5, max_pages=5 * pps, max_pages_per_seq=pps, kernel=B.KERNEL_TENSOR)
    seqs = [0, 1, 2, 3, 4]
    p.open(seqs)
    for s_, n in zip(seqs, (2100, 2049, 2111, 2050, 2064)):     # 17 tiles each: 85 tiles, 43 pairs
        p.prefill([s_], n)
    _check_step(p.decode_step(seqs, 0), "bf16", "fused clusters")


@pytest.mark.parametrize("shape", ["group2_narrow", "group4_wide", "group3_odd"])
def test_tensor_kernel_variants_walk_several_pairs(shape):
    """The tensor-core kernel is built in four variants (query groups of more than two heads or not; hidden
    layers of one 256-column chunk or more).  The two paper shapes take two of them; these shapes take the
    others, with more tile pairs than clusters so that a cluster walks several pairs (queries and tile
    positions of the next pair fetched ahead, parameter blocks kept, probability buffers handed back)."""
    if shape == "group2_narrow":     # 8 query / 4 KV heads, hidden 192: one chunk, CUDA-core attention products
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, n_q_heads=8, n_kv_heads=4, latent_full=128, batch=9,
                         cached_tokens=0, decode_steps=1, reuse_frac=0.25)
    elif shape == "group4_wide":     # 32 query / 8 KV heads, hidden 384: two chunks, tensor-op attention products
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, n_q_heads=32, n_kv_heads=8, latent_full=256, batch=9,
                         cached_tokens=0, decode_steps=1, reuse_frac=0.25)
    else:                            # 6 query / 2 KV heads: a group of three (padded inside the 8-wide operand)
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, n_q_heads=6, n_kv_heads=2, latent_full=64, batch=9,
                         cached_tokens=0, decode_steps=1, reuse_frac=0.5)
    pps = 34
    p = Pair(w, max_seqs=9, max_pages=9 * pps, max_pages_per_seq=pps, kernel=B.KERNEL_TENSOR)
    seqs = list(range(9))
    p.open(seqs)
    for s_, n in zip(seqs, (2100, 2049, 2111, 2050, 2064, 2051, 2172, 2090, 2055)):   # 17 tiles each: 77 pairs
        p.prefill([s_], n)
    assert all(p.s.ctx.layer_kernel(l) == B.KERNEL_TENSOR for l in range(w.n_layers))
    _check_step(p.decode_step(seqs, 0), "bf16", shape)


@pytest.mark.parametrize("storage", ["bf16", "f32"])
def test_many_short_sequences_merge_one_warp_per_row(storage):
    """512 (sequence, query head) rows of at most three tiles: the tile partials and the current token are merged
    by the one-warp-per-row kernel (fewer rows or longer sequences take the CTA-per-row kernel of the other tests).
    Lengths include 0 (current token only) and exact tile multiples."""
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, batch=16, cached_tokens=0, decode_steps=1, reuse_frac=0.25,
                     storage=storage)
    p = Pair(w, max_seqs=16, max_pages=16 * 6, max_pages_per_seq=6)
    seqs = list(range(16))
    p.open(seqs)
    for s_, n in zip(seqs, (0, 1, 127, 128, 129, 256, 300, 64, 5, 200, 257, 31, 33, 255, 90, 130)):
        if n:
            p.prefill([s_], n)
    _check_step(p.decode_step(seqs, 0), storage, f"warp merge {storage}")
    _check_step(p.decode_step(seqs, 1, include_current=False), storage, f"warp merge, cached only, {storage}")


@pytest.mark.parametrize("head_dim", [32, 128])
def test_other_head_widths_take_the_generic_kernels(head_dim):
    """Head widths other than 64 run on the generic kernels (fp32 and bf16 storage); 128 exercises the merge
    kernels' upper channel half, 32 their idle lanes.  One sequence is long enough (33 tiles) for the
    CTA-per-row merge, the others take the warp-per-row one."""
    for storage in ("f32", "bf16"):
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=head_dim,
                         latent_full=head_dim, batch=2, cached_tokens=0, decode_steps=1, reuse_frac=0.5,
                         storage=storage)
        for lens in ((200, 1), (4200, 130)):
            pps = (max(lens) + 2 + w.page_tokens - 1) // w.page_tokens
            p = Pair(w, max_seqs=2, max_pages=2 * pps, max_pages_per_seq=pps)
            p.open([0, 1])
            for s_, n in zip((0, 1), lens):
                p.prefill([s_], n)
            _check_step(p.decode_step([0, 1], 0), storage, f"head_dim {head_dim} {storage} {lens}")


def test_fp32_stack_with_reuse_generic():
    """fp32 mode on a multi-layer stack with chains of reuse; 1e-4 absolute."""
    w = synth.scaled(synth.CONFIGS["c2"], n_layers=4, batch=2, storage="f32", reuse_frac=0.5)
    p = Pair(w, max_seqs=2, max_pages=8, max_pages_per_seq=4)
    p.open([0, 1])
    p.prefill([0], 150)
    p.prefill([1], 33)
    p.check_latents([0, 1])
    for step in range(2):
        _check_step(p.decode_step([0, 1], step), "f32", f"step {step}")


@pytest.mark.parametrize("cfg", ["c2", "c3"])
def test_single_call_step_matches_oracle_and_the_two_calls(cfg):
    """kvcar_step_layer (tile kernel on the library's side stream beside the encoder) against the oracle, and bit
    for bit against kvcar_encode_append + kvcar_decode_attention on a twin context, over several steps (so that
    later steps read rows appended by earlier ones) and a page boundary."""
    w = synth.scaled(synth.CONFIGS[cfg], n_layers=4, batch=3, cached_tokens=0, decode_steps=3, reuse_frac=0.3)
    seqs = [0, 1, 2]
    pairs = []
    for with_oracle in (True, False):
        p = Pair(w, max_seqs=3, max_pages=24, max_pages_per_seq=8, with_oracle=with_oracle)
        p.open(seqs)
        for s_, n in zip(seqs, (383, 130, 62)):        # the third sequence crosses a page boundary at step 2
            p.prefill([s_], n)
        pairs.append(p)
    fused, split = pairs
    for step in range(3):
        a = fused.decode_step(seqs, step, fused=True)
        b = split.decode_step(seqs, step, fused=False)
        _check_step(a, "bf16", f"single call, step {step}")
        for l in a:
            assert np.array_equal(a[l][0], b[l][0]), (step, l)
    fused.check_latents(seqs)


def test_host_buffer_entry_point_matches_device_entry_points():
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, batch=2, reuse_frac=0.25)
    p = Pair(w, max_seqs=2, max_pages=8, max_pages_per_seq=4)
    seqs = [0, 1]
    p.open(seqs)
    p.prefill(seqs, 100)
    dt = p.s.dtype
    for l in range(w.n_layers):
        k = np.stack([synth.make_kv(w, l, K, s, 100, 1) for s in seqs])
        v = np.stack([synth.make_kv(w, l, V, s, 100, 1) for s in seqs])
        q = np.stack([synth.make_q(w, l, s, 0) for s in seqs])
        hk = torch.from_numpy(k).to(dt).pin_memory(); hv = torch.from_numpy(v).to(dt).pin_memory()
        hq = torch.from_numpy(q).to(dt).pin_memory()
        ho = torch.empty_like(hq).pin_memory()
        p.s.ctx.step_layer_host(l, seqs, hk.data_ptr(), hv.data_ptr(), hq.data_ptr(), ho.data_ptr(),
                                B.INCLUDE_CURRENT_EXACT, p.s.stream())
        p.s.ctx.sync_status(p.s.stream())
        p.o.encode_append(l, seqs, 1, k, v)
        ref = p.o.decode_attention(l, seqs, q)
        assert_close(ho.float().numpy().astype(np.float64), ref, "bf16", f"host entry layer {l}")


def test_errors_leave_state_untouched():
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=1, batch=1, reuse_frac=0.0)
    p = Pair(w, max_seqs=2, max_pages=2, max_pages_per_seq=2, with_oracle=False)
    p.open([0, 1])
    p.prefill([0], 64)
    big = torch.zeros(1, 100, w.kv_width, dtype=p.s.dtype, device="cuda")
    with pytest.raises(B.KvcarError) as e:      # 100 more tokens need 2 pages, 1 is left
        p.s.ctx.encode_append(0, [0], 100, big.data_ptr(), big.data_ptr(), p.s.stream())
    assert e.value.status == 3
    assert p.s.ctx.seq_len(0) == 64
    p.s.ctx.reserve([1], 64)                    # the last page is still available
    with pytest.raises(B.KvcarError) as e:
        p.s.ctx.decode_attention(0, [5], big.data_ptr(), big.data_ptr(), 0, p.s.stream())
    assert e.value.status == 1


def test_device_side_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """A bounded device-side wait that nothing completes: the kernel gives up after its limit (1 ms here), records a
    code in the status word and returns; kvcar_sync_status reports KVCAR_ERR_DEVICE_TIMEOUT exactly once, and the
    next decode on the same context is correct.  Nothing traps, faults or waits without a limit."""
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, batch=2, reuse_frac=0.25)
    p = Pair(w, max_seqs=2, max_pages=8, max_pages_per_seq=4)
    p.open([0, 1])
    p.prefill([0], 140)
    p.prefill([1], 65)
    p.s.ctx.debug_expire_wait(1_000_000, p.s.stream())
    with pytest.raises(B.KvcarError) as e:
        p.s.ctx.sync_status(p.s.stream())
    assert e.value.status == 7 and "0x7e57" in str(e.value)
    p.s.ctx.sync_status(p.s.stream())            # the word was cleared: reported once
    _check_step(p.decode_step([0, 1], 0), "bf16", "after a timed-out wait")


@pytest.mark.parametrize("cfg,quant", [("c2", False), ("c3", False), ("c2", True)])
def test_guard_regions_and_device_tables_survive_prefill_and_decode(cfg, quant):
    """Stand-in for a memory checker: 256 guard bytes behind every pool region (K and V pools, int8 row parameters,
    current-token rows) keep their fill through bulk and per-token encoding, decode steps on full and ragged
    pages, and a sequence that fills its last reserved page to the end; the device page table and lengths equal the
    allocator's.  A byte planted by the test just behind layer 0's K pool is then found and located."""
    w = synth.scaled(synth.CONFIGS[cfg], n_layers=3, batch=3, reuse_frac=0.25)
    p = Pair(w, max_seqs=3, max_pages=9, max_pages_per_seq=3, latent_quant=quant)
    p.open([0, 1, 2])
    p.prefill([0], 3 * 64 - 1)          # one step short of the end of its last page
    p.prefill([1], 65)
    p.prefill([2], 1)
    assert p.s.ctx.debug_check(p.s.stream()) == (0, 0, -1)
    p.decode_step([0, 1, 2], 0)         # sequence 0 now ends exactly at the end of the pool rows reserved for it
    assert p.s.ctx.debug_check(p.s.stream()) == (0, 0, -1)
    off, pitch, width = p.s.ctx.pool_layout(0, 0)
    rows = p.s.ctx.cfg.max_pages * p.s.ctx.cfg.page_tokens
    guard = (off + rows * pitch + 255) // 256 * 256
    base = p.s._aligned(p.s.pool) - p.s.pool.data_ptr()
    torch.cuda.synchronize()
    assert int(p.s.pool[base + guard + 7]) == 0xA5
    p.s.pool[base + guard + 7] = 0
    torch.cuda.synchronize()
    st, what, where = p.s.ctx.debug_check(p.s.stream())
    assert (st, what, where) == (8, 1, guard + 7)
    p.s.pool[base + guard + 7] = 0xA5
    torch.cuda.synchronize()
    assert p.s.ctx.debug_check(p.s.stream()) == (0, 0, -1)


@pytest.mark.parametrize("cfg", ["c2", "c3"])
def test_int8_latent_rows_match_the_oracle(cfg):
    """Sec. "Quantization" on top of the autoencoders (Table 5's combination): every cached latent row is stored
    as int8 codes with its own scale and zero-point (Eq. 4) and restored before the decoder.  Cached rows are
    compared as restored values (one code step at most, almost all equal), attention outputs at the bf16
    tolerance, bytes per token exactly."""
    w = synth.scaled(synth.CONFIGS[cfg], batch=3, cached_tokens=0, decode_steps=2)
    p = Pair(w, max_seqs=4, max_pages=16, max_pages_per_seq=6, latent_quant=True)
    seqs = [2, 0, 3]
    p.open(seqs)
    p.prefill([2], 200)
    p.prefill([0], 131)
    p.prefill([3], 1)
    p.check_latents(seqs)
    for step in range(2):
        _check_step(p.decode_step(seqs, step), "bf16", f"int8 step {step}")
    p.check_latents(seqs)
    comp, full = p.s.ctx.cache_bytes_per_token()
    assert (comp, full) == p.o.cache_bytes_per_token()
    plain = Pair(w, max_seqs=1, max_pages=1, max_pages_per_seq=1, with_oracle=False)
    assert comp < 0.55 * plain.s.ctx.cache_bytes_per_token()[0]


@pytest.mark.parametrize("shape", ["gpt2", "group2_narrow", "tinyllama"])
def test_absorbed_last_layer_on_both_sides_matches_the_oracle(shape):
    """KVCAR_ABSORBED | KVCAR_ABSORBED_V: the V side too - a tile hands on sum_t p_t a_t (m values per query head) and
    W4_h is applied once per sequence and head when the tiles are merged; no restored K or V row is ever formed.
    Same tolerance as the plain form; ragged lengths, reuse (several V sources per layer), two steps, and the
    output must also agree with the plain form of the same context."""
    if shape == "gpt2":            # 12 heads, hidden 576: nine slabs, the last feature chunk repeats a slab
        w = synth.scaled(synth.CONFIGS["c2"], n_layers=3, batch=5, cached_tokens=0, decode_steps=2, reuse_frac=0.25)
    elif shape == "tinyllama":     # 32 query / 4 KV heads (two 32-column blocks per chunk), hidden 192
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=3, batch=5, cached_tokens=0, decode_steps=2, reuse_frac=0.25)
    else:                          # 8 query / 4 KV heads, hidden 192: three slabs
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=3, n_q_heads=8, n_kv_heads=4, latent_full=128, batch=5,
                         cached_tokens=0, decode_steps=2, reuse_frac=0.25)
    pps = 34
    p = Pair(w, max_seqs=5, max_pages=5 * pps, max_pages_per_seq=pps, kernel=B.KERNEL_TENSOR)
    seqs = [0, 1, 2, 3, 4]
    p.open(seqs)
    for s_, n in zip(seqs, (2100, 2049, 2111, 2050, 2064)):     # 17 tiles each: 85 tiles, 43 pairs
        p.prefill([s_], n)
    for step in range(2):
        res = p.decode_step(seqs, step, absorbed="kv")
        _check_step(res, "bf16", f"absorbed K and V {shape} step {step}")
    # against the plain form on the same cache (one more layer call each way, no append)
    q = np.stack([synth.make_q(w, 1, s_, 7) for s_ in seqs])
    got_a, _, _ = p.attention(1, seqs, q, absorbed="kv")
    got_p, ref, rows = p.attention(1, seqs, q)
    assert_close(got_a[rows], ref, "bf16", "absorbed K and V, layer 1")
    assert np.max(np.abs(got_a - got_p)) < 2e-2
    assert np.max(np.abs(got_a - got_p)) > 0.0   # the other form did run


@pytest.mark.parametrize("shape", ["gpt2", "tinyllama", "group2_narrow"])
def test_absorbed_last_layer_matches_the_oracle(shape):
    """KVCAR_ABSORBED: a head's scores are taken as a.(W4_h^T q) + q.b4_h from the activated hidden vectors, the
    restored K rows are never formed (the decoder ends in a bare fully connected layer, Sec. "Network Architecture").
    Same result as the plain form up to rounding: compared with the oracle at the usual tolerance on grids large
    enough for the form to be taken, with reuse (several source layers per layer), and the launch counter shows that
    the operand kernel ran."""
    if shape == "gpt2":            # 12 heads, hidden 576 (three chunks), CUDA-core attention products
        w = synth.scaled(synth.CONFIGS["c2"], n_layers=3, batch=5, cached_tokens=0, decode_steps=2, reuse_frac=0.25)
    elif shape == "tinyllama":     # 32 query / 4 KV heads, hidden 192, tensor-op attention products
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=3, batch=5, cached_tokens=0, decode_steps=2, reuse_frac=0.25)
    else:                          # 8 query / 4 KV heads
        w = synth.scaled(synth.CONFIGS["c3"], n_layers=3, n_q_heads=8, n_kv_heads=4, latent_full=128, batch=5,
                         cached_tokens=0, decode_steps=2, reuse_frac=0.25)
    pps = 34
    p = Pair(w, max_seqs=5, max_pages=5 * pps, max_pages_per_seq=pps, kernel=B.KERNEL_TENSOR)
    seqs = [0, 1, 2, 3, 4]
    p.open(seqs)
    for s_, n in zip(seqs, (2100, 2049, 2111, 2050, 2064)):     # 17 tiles each: 85 tiles, 43 pairs
        p.prefill([s_], n)
    for step in range(2):
        before = p.s.ctx.launch_count()
        res = p.decode_step(seqs, step, absorbed=True)
        # per layer: two encoder launches, the operand kernel, the tile kernel, the combine kernel (+ table updates)
        assert p.s.ctx.launch_count() - before >= 5 * w.n_layers
        _check_step(res, "bf16", f"absorbed {shape} step {step}")
    # the flag is a no-op where the form is not taken (a grid small enough for the K/V split): same tolerance
    w2 = synth.scaled(w, batch=2)
    p2 = Pair(w2, max_seqs=2, max_pages=8, max_pages_per_seq=4, kernel=B.KERNEL_TENSOR)
    p2.open([0, 1])
    p2.prefill([0], 200)
    p2.prefill([1], 130)
    _check_step(p2.decode_step([0, 1], 0, absorbed=True), "bf16", f"absorbed flag on a small grid, {shape}")

