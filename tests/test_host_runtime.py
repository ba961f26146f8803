"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol,
and its integer bookkeeping (reuse resolution, page allocation, accounting)
matches the oracle bit for bit.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import kvcar_synth as synth
from oracle.kvcar_oracle import K, V, KVCAROracle
from paper_2512_06727_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "kvcar.h")).read()
    declared = sorted(set(re.findall(r"\b(kvcar_[a-z_0-9]+)\s*\(", header)))
    assert len(declared) >= 20
    lib = B.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == declared


def _pair(w, src_k, src_v, max_seqs=6, max_pages=40, mpps=12, compressed_layers=None):
    o = KVCAROracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, max_seqs, max_pages, w.storage)
    c = B.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, max_seqs, max_pages, mpps,
                  B.BF16 if w.storage == "bf16" else B.F32)
    o.set_reuse_map(src_k, src_v)
    c.set_reuse_map(src_k, src_v)
    aes = synth.make_stack_autoencoders(w, src_k, src_v, layers=compressed_layers)
    for (l, which), ae in aes.items():
        o.set_autoencoder(l, which, ae)
        c.set_autoencoder(l, which, ae)
    return o, c


@pytest.mark.parametrize("name", ["c2", "c3"])
def test_resolve_matches_oracle_on_benchmark_maps(name):
    w = synth.CONFIGS[name]
    src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    src_v = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed + 100)  # K and V differ
    o, c = _pair(w, src, src_v)
    for l in range(w.n_layers):
        for h in range(w.n_kv_heads):
            for which in (K, V):
                assert c.debug_resolve(l, h, which) == o.resolve(l, h, which)
    assert c.cache_bytes_per_token() == o.cache_bytes_per_token()


def test_resolve_random_chains():
    rng = np.random.default_rng(0)
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=9, n_kv_heads=4, n_q_heads=8)
    for trial in range(20):
        src_k = -np.ones((9, 4), np.int32)
        src_v = -np.ones((9, 4), np.int32)
        for s in (src_k, src_v):
            mask = rng.random((8, 4)) < 0.6
            s[1:][mask] = rng.integers(0, 4, size=int(mask.sum()))   # arbitrary head of the layer below
        o = KVCAROracle(9, 8, 4, 64, 64, 1, 1)
        c = B.Context(9, 8, 4, 64, 64, 1, 1, 1, B.F32)
        o.set_reuse_map(src_k.reshape(-1), src_v.reshape(-1))
        c.set_reuse_map(src_k.reshape(-1), src_v.reshape(-1))
        for l in range(9):
            for h in range(4):
                for which in (K, V):
                    assert c.debug_resolve(l, h, which) == o.resolve(l, h, which)


def test_reuse_map_validation():
    c = B.Context(3, 4, 2, 64, 64, 1, 1, 1, B.F32)
    with pytest.raises(B.KvcarError) as e:
        c.set_reuse_map([0, -1, -1, -1, -1, -1], [-1] * 6)
    assert e.value.status == 1
    with pytest.raises(B.KvcarError):
        c.set_reuse_map([-1, -1, 2, -1, -1, -1], [-1] * 6)
    with pytest.raises(B.KvcarError):
        c.set_reuse_map([-1, -1, -2, -1, -1, -1], [-1] * 6)
    c.set_reuse_map([-1, -1, 1, 0, 1, 1], [-1] * 6)
    ae = synth.make_autoencoder(128, 96, 64, 0, 0, 0)
    c.set_autoencoder(0, 0, ae)
    with pytest.raises(B.KvcarError) as e:      # layer 2 stores no K head at all: in_dim 128 is wrong
        c.set_autoencoder(2, 0, ae)
    assert e.value.status == 1
    with pytest.raises(B.KvcarError) as e:      # map is frozen once an autoencoder depends on it
        c.set_reuse_map([-1] * 6, [-1] * 6)
    assert e.value.status == 2


def test_page_allocator_matches_oracle():
    w = synth.scaled(synth.CONFIGS["c3"], n_layers=2, page_tokens=16)
    src = np.full(2 * w.n_kv_heads, -1, np.int32)
    o, c = _pair(w, src, src, max_seqs=6, max_pages=40, mpps=12)
    rng = np.random.default_rng(1)
    open_seqs = []
    for step in range(400):
        r = rng.random()
        if r < 0.15 and len(open_seqs) < 6:
            s = int(rng.choice([i for i in range(6) if i not in open_seqs]))
            o.seq_open(s); c.seq_open(s); open_seqs.append(s)
        elif r < 0.25 and open_seqs:
            s = open_seqs.pop(int(rng.integers(len(open_seqs))))
            o.seq_close(s); c.seq_close(s)
        elif open_seqs:
            k = int(rng.integers(1, len(open_seqs) + 1))
            seqs = [int(x) for x in rng.permutation(open_seqs)[:k]]
            n = int(rng.integers(1, 40))
            if any(o.seq_len[s] + n > 12 * 16 for s in seqs):
                with pytest.raises(B.KvcarError) as e:      # longer than max_pages_per_seq allows
                    c.reserve(seqs, n)
                assert e.value.status == 3
                continue
            try:
                o.reserve(seqs, n)
            except MemoryError:
                with pytest.raises(B.KvcarError) as e:      # pool exhausted: refused, nothing taken
                    c.reserve(seqs, n)
                assert e.value.status == 3
                continue
            c.reserve(seqs, n)
            o.advance(seqs, n); c.advance(seqs, n)
        for s in open_seqs:
            assert c.seq_len(s) == o.seq_len[s]
            for t in range(0, o.seq_len[s], 7):
                assert c.debug_locate(s, t) == o.locate(s, t)
            if o.seq_len[s]:
                assert c.debug_locate(s, o.seq_len[s] - 1) == o.locate(s, o.seq_len[s] - 1)


def test_accounting_and_layout():
    w = synth.CONFIGS["c2"]
    src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    o, c = _pair(w, src, src, compressed_layers=list(range(10)))
    assert c.cache_bytes_per_token() == o.cache_bytes_per_token()
    pool_b, w_b, ws_b = c.required_bytes()
    rows = 40 * 64
    total = 0
    last_end = 0
    for l in range(w.n_layers):
        for which in (K, V):
            off, pitch, width = c.pool_layout(l, which)
            assert width == o.stored_width(l, which) and pitch == width * 2
            assert off % 256 == 0 and off >= last_end
            last_end = off + rows * pitch
            total += rows * pitch
    assert pool_b >= total
    # work model: no reuse, GPT-2-small shape -> 1536 latent bytes and 2 654 208 + 3072 flops per token-layer
    w1 = synth.CONFIGS["c1"]
    none = np.full(w1.n_kv_heads, -1, np.int32)
    o1, c1 = _pair(synth.scaled(w1, storage="bf16"), none, none)
    assert c1.layer_work_per_token(0) == (1536.0, 2654208.0 + 3072.0)


def test_int8_latent_rows_accounting_and_layout():
    """int8 latent rows (Sec. "Quantization", Eq. 4): one byte per element plus 8 bytes of scale and zero-point
    per cached row and (layer, K/V); the library's bytes per token equal the oracle's, the codes' row pitch is the
    width in bytes and the parameter array follows the codes, 256-byte aligned."""
    for name in ("c2", "c3"):
        w = synth.CONFIGS[name]
        src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
        o = KVCAROracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, 6, 40, "int8")
        c = B.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, 6, 40, 12, B.BF16, 1)
        o.set_reuse_map(src, src)
        c.set_reuse_map(src, src)
        for (l, which), ae in synth.make_stack_autoencoders(w, src, src).items():
            o.set_autoencoder(l, which, ae)
            c.set_autoencoder(l, which, ae)
        assert c.cache_bytes_per_token() == o.cache_bytes_per_token()
        rows = 40 * w.page_tokens
        for l in range(w.n_layers):
            for which in (K, V):
                off, pitch, width = c.pool_layout(l, which)
                assert width == o.stored_width(l, which) and pitch == width
                if width:
                    par = c.pool_quant_layout(l, which)
                    assert par % 256 == 0 and par >= off + rows * pitch
    # a stack with uncompressed stored rows cannot take int8 latent rows: bind refuses, nothing is launched
    w = synth.CONFIGS["c2"]
    c = B.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, 2, 4, 2, B.BF16, 1)
    with pytest.raises(B.KvcarError) as e:
        c.bind_memory(256, 1 << 20, 512, 1 << 20, 768, 1 << 20, 0)
    assert e.value.status == 5


def test_library_accounting_reproduces_the_printed_percentages():
    """The library's own kvcar_cache_bytes_per_token, driven through the C ABI, against the cache reductions the paper
    prints (Tables 2, 3 and 4; the records and their citations are in tests/golden/paper_accounting.txt)."""
    golden = os.path.join(ROOT, "tests", "golden", "paper_accounting.txt")
    seen = 0
    for line in open(golden):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        kind, params, printed, cite = [p_.strip() for p_ in line.split("|")]
        if kind.startswith("eq3"):
            continue
        kv = dict(p_.split("=") for p_ in params.split())
        layers, heads, hd = int(kv["layers"]), int(kv["heads"]), 64
        src = [np.full((layers, heads), -1, np.int32), np.full((layers, heads), -1, np.int32)]
        for which, key in ((K, "k_heads"), (V, "v_heads")):
            n = kv.get(key, "0")
            if n == "all":
                src[which][1::2, :] = np.arange(heads)        # every second layer reads the layer below
            else:
                cand = [(l, h) for l in range(1, layers, 2) for h in range(heads)]
                for l, h in cand[:int(n)]:
                    src[which][l, h] = h
        c = B.Context(layers, heads, heads, hd, 64, 1, 1, 1, B.BF16)
        c.set_reuse_map(src[K].reshape(-1), src[V].reshape(-1))
        ratio = float(kv.get("ratio", 1.0))
        for l in range(int(kv.get("compressed", 0))):
            for which in (K, V):
                n_stored = int((src[which][l] < 0).sum())
                if n_stored:
                    i, m, d = synth.ae_dims(n_stored, hd, int(hd * ratio))
                    c.set_autoencoder(l, which, synth.make_autoencoder(i, m, d, 0, l, which, storage="bf16"))
        comp, full = c.cache_bytes_per_token()
        assert abs(100.0 * (1.0 - comp / full) - float(printed)) < 0.1, (cite, comp, full)
        seen += 1
    assert seen == 12


def test_launching_calls_need_bound_memory():
    c = B.Context(1, 4, 2, 64, 64, 2, 4, 2, B.BF16)
    c.seq_open(0)
    with pytest.raises(B.KvcarError) as e:
        c.encode_append(0, [0], 1, 256, 256)
    assert e.value.status == 2
    with pytest.raises(B.KvcarError) as e:
        c.decode_attention(0, [0], 256, 256)
    assert e.value.status == 2
    with pytest.raises(B.KvcarError):
        B.Context(1, 5, 2, 64, 64, 2, 4, 2, B.BF16)      # query heads not a multiple of KV heads


def test_reuse_map_from_l1_matches_oracle_bit_for_bit():
    """Alg. 2's choice of reused heads is integer work on the host: the library's table equals the oracle's for
    random distances (with planted ties) at every count, and bad arguments are refused."""
    from oracle import kvcar_oracle as orc
    rng = np.random.default_rng(11)
    for (L, H) in ((12, 12), (22, 4), (2, 1)):
        dist = rng.random((L - 1, H)).astype(np.float32)
        if dist.size > 3:
            dist.flat[3] = dist.flat[0]          # ties: the lower (layer, head) goes first
            dist.flat[-1] = dist.flat[0]
        for n_reuse in sorted({0, 1, dist.size // 4, dist.size}):
            got = B.reuse_map_from_l1(dist.ravel().tolist(), L, H, n_reuse)
            want = orc.reuse_map_from_l1(dist.astype(np.float64), n_reuse)
            assert got == want.tolist(), (L, H, n_reuse)
            assert sum(1 for v in got if v >= 0) == n_reuse and all(v == -1 for v in got[:H])
    with pytest.raises(B.KvcarError):
        B.reuse_map_from_l1([0.1, 0.2], 2, 2, 3)              # more heads than there are
    with pytest.raises(B.KvcarError):
        B.reuse_map_from_l1([0.1, float("nan")], 2, 2, 1)
    # size query and argument checks of the distance call need no GPU
    assert B.head_l1_scratch_bytes(12, 12, 8192) == (8192 // 8) * 11 * 12 * 4
    with pytest.raises(B.KvcarError):
        B.head_l1_scratch_bytes(1, 12, 8192)                  # one layer has no layer below
    with pytest.raises(B.KvcarError):
        B.head_l1_distance(12, 12, 60, B.BF16, 16, 8, 16, 1 << 20, 16)   # a 60-wide head is not whole 16-byte chunks


def test_trace_report_reads_synthetic_stamps(capsys):
    """The time-stamp reader of the tensor kernel (python -m paper_2512_06727_b200.trace) on hand-made records: two
    jobs of the issuer (a hidden chunk of two slabs, a head group of one) and their epilogues."""
    from paper_2512_06727_b200 import trace
    iss = [(100, 0x11), (150, 0x30), (400, 0x31), (500, 0x30), (800, 0x31), (900, 0x19),
           (1000, 0x12), (1100, 0x30), (1400, 0x31), (1500, 0x19)]
    ep = [(50, 0x40), (950, 0x41), (1950, 0x43), (2000, 0x50), (2100, 0x51), (2200, 0x52), (2600, 0x53)]
    trace.report({"0.0": [], "0.1": [], "0.2": iss, "0.3": ep, "1.0": [], "1.1": [], "1.2": [], "1.3": []}, 5)
    out = capsys.readouterr().out
    assert "issuer: 2 jobs, 3 slabs in 1400 cycles; waiting 250, issuing 850, between jobs 100" in out
    assert "hidden chunk jobs: 1, mean 800 cycles, 400 per slab" in out
    assert "head group jobs: 1, mean 500 cycles, 500 per slab" in out
    assert "epilogue, hidden chunk: 1 jobs, mean wait 900, mean work 1000 cycles" in out
    trace.report({"0.2": [], "0.3": []}, 5)
    assert "no stamps" in capsys.readouterr().out



def test_status_codes_of_the_header_match_the_binding():
    """Every KVCAR_ERR_* / KVCAR_OK of include/kvcar.h has the same number and name in the Python binding (a status the
    binding cannot name would be raised as a bare number)."""
    import os
    import re
    from paper_2512_06727_b200 import binding as B
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "include", "kvcar.h")).read()
    body = text[text.index("KVCAR_OK = 0"):]
    body = body[:body.index("}")]
    codes = {int(v): k for k, v in re.findall(r"KVCAR_(?:ERR_)?([A-Z_]+)\s*=\s*(\d+)", body)}
    assert codes == B.STATUS_NAMES, (codes, B.STATUS_NAMES)
