"""GPU parity of the Alg. 2 statistic (mean absolute difference between a head and the same head one layer
down) against the CPU oracle, through the C ABI, and the reuse table chosen from it."""
import numpy as np
import pytest
import torch

from oracle import kvcar_oracle as orc
from paper_2512_06727_b200 import binding as B

pytestmark = pytest.mark.gpu


def _activations(n_layers, n_rows, hkv, hd, seed, dtype):
    """Layers that drift away from the layer below by a head- and layer-specific amount, so that the distances
    differ by head (seeded; on the storage grid)."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    x = torch.empty(n_layers, n_rows, hkv * hd, dtype=torch.float32)
    x[0] = torch.randn(n_rows, hkv * hd, generator=g)
    for l in range(1, n_layers):
        sigma = torch.rand(hkv, generator=g).repeat_interleave(hd) * 0.8 + 0.05
        x[l] = x[l - 1] + sigma * torch.randn(n_rows, hkv * hd, generator=g)
    return x.to(dtype)


def _run(x, hkv, hd, storage):
    n_layers, n_rows, _ = x.shape
    dev = x.cuda().contiguous()
    nbytes = B.head_l1_scratch_bytes(n_layers, hkv, n_rows)
    scratch = torch.full((nbytes // 4 + 4,), float("nan"), device="cuda")      # contents must not matter
    dist = torch.full((n_layers - 1, hkv), float("nan"), device="cuda")
    B.head_l1_distance(n_layers, hkv, hd, storage, dev.data_ptr(), n_rows, scratch.data_ptr(), nbytes, dist.data_ptr(),
                       torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return dist.cpu().numpy()


@pytest.mark.parametrize("case", [
    ("bf16", 12, 1000, 12, 64),      # GPT-2-small shape, rows not a multiple of a CTA's 21
    ("bf16", 22, 777, 4, 64),        # TinyLLaMA shape (64 rows per CTA, ragged tail)
    ("f32", 3, 50, 3, 20),           # odd head width in fp32, 85 rows per CTA: a single partly filled CTA
    ("bf16", 2, 1, 16, 128),         # one row, the widest configuration
], ids=lambda c: f"{c[0]}-L{c[1]}-R{c[2]}-H{c[3]}x{c[4]}")
def test_head_l1_distance_matches_oracle(case):
    name, n_layers, n_rows, hkv, hd = case
    dtype, storage = (torch.bfloat16, B.BF16) if name == "bf16" else (torch.float32, B.F32)
    x = _activations(n_layers, n_rows, hkv, hd, seed=n_layers * 1000 + n_rows, dtype=dtype)
    got = _run(x, hkv, hd, storage)
    want = orc.head_l1_distance(x.float().numpy().astype(np.float64), hkv)
    # fp32 sums of n_rows * hd non-negative terms in a fixed order: relative error well below 1e-5
    np.testing.assert_allclose(got, want, rtol=2e-5, atol=1e-7)
    again = _run(x, hkv, hd, storage)
    assert np.array_equal(got, again)                                          # fixed summation order
    # the reuse table chosen from the GPU's distances equals the oracle's choice from the same numbers
    n_reuse = got.size // 4
    table = B.reuse_map_from_l1(got.ravel().tolist(), n_layers, hkv, n_reuse)
    assert table == orc.reuse_map_from_l1(got.astype(np.float64), n_reuse).tolist()


def test_scratch_too_small_is_refused():
    x = torch.zeros(2, 64, 4 * 64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4, device="cuda")
    scratch = torch.zeros(64, device="cuda")
    with pytest.raises(B.KvcarError) as e:
        B.head_l1_distance(2, 4, 64, B.BF16, x.data_ptr(), 64, scratch.data_ptr(), 4, out.data_ptr(), 0)
    assert e.value.status == 4          # KVCAR_ERR_WORKSPACE


def test_reuse_table_from_distances_drives_the_cache():
    """Alg. 2 end to end on synthetic activations: distances on the GPU, the closest heads chosen by the library,
    the table handed to a cache context, and a decode step over that cache checked against the oracle, which gets
    the table chosen by ITS OWN distance and choice functions (the two tables must be identical)."""
    import kvcar_synth as synth
    from kvcar_harness import Pair, assert_close
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=4, batch=2, cached_tokens=0, decode_steps=1, reuse_frac=0.0)
    hkv, hd, L = w.n_kv_heads, w.head_dim, w.n_layers
    tables = {}
    for which, seed in (("k", 21), ("v", 22)):
        x = _activations(L, 600, hkv, hd, seed=seed, dtype=torch.bfloat16)
        got = _run(x, hkv, hd, B.BF16)
        n_reuse = 5
        lib_table = B.reuse_map_from_l1(got.ravel().tolist(), L, hkv, n_reuse)
        want = orc.head_l1_distance(x.float().numpy().astype(np.float64), hkv)
        oracle_table = orc.reuse_map_from_l1(want, n_reuse).tolist()
        assert lib_table == oracle_table, which          # the distances differ by ~1e-7 relative: same ranking here
        tables[which] = np.array(lib_table, dtype=np.int32)
    assert (tables["k"] >= 0).sum() == 5 and not np.array_equal(tables["k"], tables["v"])
    p = Pair(w, max_seqs=2, max_pages=12, max_pages_per_seq=6, src_k=tables["k"], src_v=tables["v"])
    p.open([0, 1])
    p.prefill([0], 300)
    p.prefill([1], 129)
    for l, (gpu, ref, rows) in p.decode_step([0, 1], 0).items():
        assert_close(gpu[rows], ref, "bf16", f"layer {l}")
    stored = sum(len(p.o.stored_heads(l, 0)) for l in range(L))
    assert stored == L * hkv - 5                         # the five reused K heads store nothing
