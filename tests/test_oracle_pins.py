"""Pins for the CPU oracle: what the paper and the mathematics fix, checked
against code that is NOT the oracle (plain definitions retyped here, torch CPU
routines, brute-force loops, closed forms, printed values)."""
import math
import os

import numpy as np
import pytest
import torch

import kvcar_synth as synth
from oracle import kvcar_oracle as orc
from oracle.kvcar_oracle import K, V, KVCAROracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_accounting.txt")


# ---------------------------------------------------------------- helpers
def plain_sdpa(q, keys, vals):
    """Eq. 1 for one head, written out: softmax(q K^T / sqrt(d_k)) V."""
    d_k = q.shape[0]
    s = np.array([sum(q[c] * keys[j, c] for c in range(d_k)) / math.sqrt(d_k) for j in range(keys.shape[0])])
    w = np.exp(s - s.max())
    w = w / w.sum()
    return sum(w[j] * vals[j] for j in range(keys.shape[0]))


def identity_ae(width):
    eye = np.eye(width)
    one = np.ones(width)
    zero = np.zeros(width)
    bn = np.stack([one, zero, zero, one])
    return {"in_dim": width, "hidden": width, "latent": width, "leaky_slope": 1.0, "bn_eps": 0.0,
            "enc_w1": eye, "enc_b1": zero, "enc_bn": bn, "enc_w2": eye, "enc_b2": zero,
            "dec_w1": eye, "dec_b1": zero, "dec_bn": bn, "dec_w2": eye, "dec_b2": zero}


def small_stack(n_layers=3, hq=4, hkv=2, hd=8, P=4, max_seqs=3, max_pages=16, storage="exact",
                reuse=None, seed=11, lat_per_head=4, with_ae=True, slope=0.01):
    o = KVCAROracle(n_layers, hq, hkv, hd, P, max_seqs, max_pages, storage)
    src_k = np.full(n_layers * hkv, -1, np.int32)
    src_v = np.full(n_layers * hkv, -1, np.int32)
    for (which, l, h, s) in (reuse or []):
        (src_k if which == K else src_v)[l * hkv + h] = s
    o.set_reuse_map(src_k, src_v)
    if with_ae:
        for l in range(n_layers):
            for which, src in ((K, src_k), (V, src_v)):
                n = len(synth.stored_heads(src, hkv, l))
                if n:
                    i, m, d = synth.ae_dims(n, hd, lat_per_head)
                    o.set_autoencoder(l, which, synth.make_autoencoder(i, m, d, seed, l, which, leaky_slope=slope))
    return o


def fill(o, seqs, n_tokens, seed=5, steps=1):
    """prefill n_tokens, then `steps` single-token appends; returns all raw K/V fed."""
    W = o.hkv * o.hd
    g = np.random.default_rng(seed)
    fed = {}
    for s in seqs:
        o.seq_open(s)
    for l in range(o.n_layers):
        k = g.standard_normal((len(seqs), n_tokens, W))
        v = g.standard_normal((len(seqs), n_tokens, W))
        fed[(l, 0)] = (k, v)
        o.encode_append(l, seqs, n_tokens, k, v)
    o.advance(seqs, n_tokens)
    return fed, g


# ---------------------------------------------------------------- Eq. 1 special case
def test_identity_autoencoder_is_plain_attention():
    hq, hkv, hd, L = 4, 2, 8, 9
    o = KVCAROracle(1, hq, hkv, hd, 4, 2, 8, "exact")
    o.set_reuse_map([-1] * hkv, [-1] * hkv)
    o.set_autoencoder(0, K, identity_ae(hkv * hd))
    o.set_autoencoder(0, V, identity_ae(hkv * hd))
    g = np.random.default_rng(0)
    k = g.standard_normal((1, L, hkv * hd)); v = g.standard_normal((1, L, hkv * hd))
    o.seq_open(0)
    o.encode_append(0, [0], L, k, v)
    o.advance([0], L)
    kc = g.standard_normal((1, 1, hkv * hd)); vc = g.standard_normal((1, 1, hkv * hd))
    o.encode_append(0, [0], 1, kc, vc)
    q = g.standard_normal((1, hq, hd))
    out = o.decode_attention(0, [0], q, include_current=True)
    kk = np.vstack([k[0], kc[0]]); vv = np.vstack([v[0], vc[0]])
    for qh in range(hq):
        gidx = qh // (hq // hkv)
        ref = plain_sdpa(q[0, qh], kk[:, gidx * hd:(gidx + 1) * hd], vv[:, gidx * hd:(gidx + 1) * hd])
        assert np.max(np.abs(out[0, qh] - ref)) < 1e-12
    # third opinion: torch's fp64 SDPA with grouped KV heads expanded
    tq = torch.tensor(q[0]).unsqueeze(1)                                 # [hq,1,hd]
    tk = torch.tensor(kk).reshape(-1, hkv, hd).permute(1, 0, 2).repeat_interleave(hq // hkv, 0)
    tv = torch.tensor(vv).reshape(-1, hkv, hd).permute(1, 0, 2).repeat_interleave(hq // hkv, 0)
    tref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).squeeze(1).numpy()
    assert np.max(np.abs(out[0] - tref)) < 1e-12
    # with an identity autoencoder, "cached only after advance" equals "cached + exact current"
    o.advance([0], 1)
    out_b = o.decode_attention(0, [0], q, include_current=False)
    assert np.max(np.abs(out_b - out)) < 1e-12


# ---------------------------------------------------------------- autoencoder vs library routines
@pytest.mark.parametrize("trivial_bn", [False, True])
def test_autoencoder_matches_torch_functional(trivial_bn):
    ae = synth.make_autoencoder(48, 36, 24, seed=3, layer=1, which=0, trivial_bn=trivial_bn)
    x = np.random.default_rng(1).standard_normal((7, 48))
    F = torch.nn.functional
    t = lambda a: torch.tensor(np.asarray(a, np.float64))

    def torch_half(inp, w1, b1, bn, w2, b2):
        a = F.linear(inp, t(w1), t(b1))
        a = F.batch_norm(a, t(bn[2]), t(bn[3]), t(bn[0]), t(bn[1]), training=False, eps=ae["bn_eps"])
        a = F.leaky_relu(a, ae["leaky_slope"])
        return F.linear(a, t(w2), t(b2))

    z_ref = torch_half(t(x), ae["enc_w1"], ae["enc_b1"], ae["enc_bn"], ae["enc_w2"], ae["enc_b2"])
    z = orc.encode(ae, x)
    assert np.max(np.abs(z - z_ref.numpy())) < 1e-12
    y_ref = torch_half(z_ref, ae["dec_w1"], ae["dec_b1"], ae["dec_bn"], ae["dec_w2"], ae["dec_b2"])
    assert np.max(np.abs(orc.decode(ae, z) - y_ref.numpy())) < 1e-12
    assert z.shape == (7, 24) and y_ref.shape == (7, 48)


def test_leaky_relu_and_bn_are_not_no_ops():
    """A dropped BN term or activation must change the result (guards the pins above
    against being vacuous)."""
    ae = synth.make_autoencoder(16, 12, 8, seed=9, layer=0, which=1)
    x = np.random.default_rng(2).standard_normal((5, 16))
    base = orc.encode(ae, x)
    lin = dict(ae, leaky_slope=1.0)
    assert np.max(np.abs(orc.encode(lin, x) - base)) > 1e-3
    nobn = dict(ae, enc_bn=np.stack([np.ones(12), np.zeros(12), np.zeros(12), np.ones(12)]))
    assert np.max(np.abs(orc.encode(nobn, x) - base)) > 1e-3


# ---------------------------------------------------------------- brute force on tiny shapes
def brute_force(n_layers, hq, hkv, hd, P, src_k, src_v, aes, fed_k, fed_v, cur_k, cur_v, q, layer, L, slope, eps):
    """The whole method for ONE sequence with explicit loops and python floats.
    fed_k[l]: [L][W] raw rows of cached tokens; cur_k[l]: [W] current rows."""
    W = hkv * hd

    def lin(x, w, b):
        return [sum(w[o][i] * x[i] for i in range(len(x))) + b[o] for o in range(len(b))]

    def half(x, w1, b1, bn, w2, b2):
        a = lin(x, w1, b1)
        a = [bn[0][j] * (a[j] - bn[2][j]) / math.sqrt(bn[3][j] + eps) + bn[1][j] for j in range(len(a))]
        a = [t if t > 0 else slope * t for t in a]
        return lin(a, w2, b2)

    def stored(src, l):
        return [h for h in range(hkv) if src[l * hkv + h] < 0]

    def root(src, l, h):
        while src[l * hkv + h] >= 0:
            h = src[l * hkv + h]
            l -= 1
        return l, h

    def rows_for(which, src, fed, cur, g):
        rl, rh = root(src, layer, g)
        heads = stored(src, rl)
        slot = heads.index(rh)
        ae = aes[(rl, which)]
        rows = []
        for t in range(L):
            x = [fed[rl][t][h * hd + c] for h in heads for c in range(hd)]
            z = half(x, ae["enc_w1"], ae["enc_b1"], ae["enc_bn"], ae["enc_w2"], ae["enc_b2"])
            y = half(z, ae["dec_w1"], ae["dec_b1"], ae["dec_bn"], ae["dec_w2"], ae["dec_b2"])
            rows.append(y[slot * hd:(slot + 1) * hd])
        rows.append([cur[rl][rh * hd + c] for c in range(hd)])
        return rows

    out = []
    for qh in range(hq):
        g = qh // (hq // hkv)
        kr = rows_for(K, src_k, fed_k, cur_k, g)
        vr = rows_for(V, src_v, fed_v, cur_v, g)
        s = [sum(q[qh][c] * kr[j][c] for c in range(hd)) / math.sqrt(hd) for j in range(L + 1)]
        mx = max(s)
        e = [math.exp(t - mx) for t in s]
        z = sum(e)
        out.append([sum(e[j] / z * vr[j][c] for j in range(L + 1)) for c in range(hd)])
    return np.array(out)


@pytest.mark.parametrize("layer", [0, 1, 2])
def test_brute_force_tiny(layer):
    n_layers, hq, hkv, hd, P, L = 3, 4, 2, 4, 2, 5
    # K: layer1 head0 <- layer0 head0 ; layer2 head0 <- layer1 head0 (chain) ; layer2 head1 <- layer1 head0 (cross index)
    # V: layer2 head1 <- layer1 head1
    reuse = [(K, 1, 0, 0), (K, 2, 0, 0), (K, 2, 1, 0), (V, 2, 1, 1)]
    o = small_stack(n_layers, hq, hkv, hd, P, 2, 8, "exact", reuse, seed=21, lat_per_head=2)
    g = np.random.default_rng(3)
    W = hkv * hd
    o.seq_open(1)
    fed_k, fed_v, cur_k, cur_v = {}, {}, {}, {}
    for l in range(n_layers):
        fed_k[l] = g.standard_normal((L, W)); fed_v[l] = g.standard_normal((L, W))
        o.encode_append(l, [1], L, fed_k[l][None], fed_v[l][None])
    o.advance([1], L)
    for l in range(n_layers):
        cur_k[l] = g.standard_normal(W); cur_v[l] = g.standard_normal(W)
        o.encode_append(l, [1], 1, cur_k[l][None, None], cur_v[l][None, None])
    q = g.standard_normal((hq, hd))
    got = o.decode_attention(layer, [1], q[None], include_current=True)[0]
    ref = brute_force(n_layers, hq, hkv, hd, P, list(o.src[K].reshape(-1)), list(o.src[V].reshape(-1)),
                      {k_: {n: (np.asarray(a, np.float64).tolist() if isinstance(a, np.ndarray) else a)
                            for n, a in v_.items()} for k_, v_ in o.ae.items()},
                      {l: fed_k[l].tolist() for l in fed_k}, {l: fed_v[l].tolist() for l in fed_v},
                      {l: cur_k[l].tolist() for l in cur_k}, {l: cur_v[l].tolist() for l in cur_v},
                      q.tolist(), layer, L, 0.01, 1e-5)
    assert np.max(np.abs(got - ref)) < 1e-12


# ---------------------------------------------------------------- reuse
def test_resolve_chains_and_slots():
    hkv = 4
    o = KVCAROracle(4, 4, hkv, 8, 4, 1, 4)
    src_k = -np.ones((4, hkv), int)
    src_k[1, 2] = 2          # l1h2 <- l0h2
    src_k[2, 2] = 2          # l2h2 <- l1h2 <- l0h2
    src_k[3, 0] = 2          # l3h0 <- l2h2 <- ... l0h2
    src_k[2, 0] = 1          # l2h0 <- l1h1 (own)
    src_k[1, 0] = 3          # l1h0 <- l0h3
    src_v = -np.ones((4, hkv), int)
    o.set_reuse_map(src_k.reshape(-1), src_v.reshape(-1))
    assert o.resolve(0, 2, K) == (0, 2, 2)
    assert o.resolve(1, 2, K) == (0, 2, 2)
    assert o.resolve(2, 2, K) == (0, 2, 2)
    assert o.resolve(3, 0, K) == (0, 2, 2)
    assert o.resolve(2, 0, K) == (1, 1, 0)     # layer 1 stores heads {1,3}: head 1 is slot 0
    assert o.resolve(1, 3, K) == (1, 3, 1)
    assert o.resolve(1, 0, K) == (0, 3, 3)
    assert o.resolve(3, 3, V) == (3, 3, 3)
    assert o.stored_heads(1, K) == [1, 3] and o.stored_heads(2, K) == [1, 3]
    with pytest.raises(ValueError):
        o.set_reuse_map([0] + [-1] * 15, [-1] * 16)        # layer 0 cannot reuse
    with pytest.raises(ValueError):
        o.set_reuse_map([-1] * 4 + [4] + [-1] * 11, [-1] * 16)  # head out of range


def test_reused_head_equals_recomputing_with_lower_layer():
    """A head of layer l that reuses layer l-1's head must give exactly what layer
    l-1's cache, decoder and current token give for that query."""
    reuse = [(K, 1, 1, 1), (V, 1, 1, 1), (K, 2, 1, 1), (V, 2, 0, 0)]
    o = small_stack(3, 4, 2, 8, 4, 2, 16, "bf16", reuse, seed=4)
    fed, g = fill(o, [0, 1], 10)
    W = o.hkv * o.hd
    for l in range(3):
        o.encode_append(l, [0, 1], 1, g.standard_normal((2, 1, W)), g.standard_normal((2, 1, W)))
    q = g.standard_normal((2, 4, 8))
    out = {l: o.decode_attention(l, [0, 1], q) for l in range(3)}
    # layer1, kv head 1 (query heads 2,3): K and V both from layer 0 head 1 -> identical to layer 0's output
    assert np.array_equal(out[1][:, 2:4], out[0][:, 2:4])
    # layer2, kv head 1: K chains to layer 0 head 1, V is layer 2's own -> must differ from layer 0 ...
    assert not np.allclose(out[2][:, 2:4], out[0][:, 2:4])
    # ... and equal a by-hand mix: softmax weights from layer-0 keys, values from layer-2's own decoder
    for s in (0, 1):
        for qh in (2, 3):
            keys = np.vstack([o.restored_rows(0, K, s)[:, 8:16], o.cur[(0, K, s)][8:16]])
            vals = np.vstack([o.restored_rows(2, V, s)[:, 0:8], o.cur[(2, V, s)][8:16]])
            # layer 2 stores V heads {1} only (head 0 is reused) -> head 1 sits in slot 0
            ref = plain_sdpa(q[s, qh], keys, vals)
            assert np.max(np.abs(out[2][s, qh] - ref)) < 1e-12
    # a reused head's own input columns are ignored: feed garbage there and nothing changes
    o2 = small_stack(3, 4, 2, 8, 4, 2, 16, "bf16", reuse, seed=4)
    fill(o2, [0, 1], 10)
    assert o2.stored_width(1, K) == 4 and o2.stored_width(0, K) == 8


def test_reuse_ignores_the_reusing_heads_input_columns():
    reuse = [(K, 1, 0, 0), (V, 1, 0, 0)]
    outs = []
    for junk in (0.0, 100.0):
        o = small_stack(2, 2, 2, 8, 4, 1, 8, "exact", reuse, seed=8)
        g = np.random.default_rng(7)
        o.seq_open(0)
        for l in range(2):
            k = g.standard_normal((1, 6, 16)); v = g.standard_normal((1, 6, 16))
            if l == 1:
                k[..., :8] += junk; v[..., :8] += junk
            o.encode_append(l, [0], 6, k, v)
        o.advance([0], 6)
        for l in range(2):
            k = g.standard_normal((1, 1, 16)); v = g.standard_normal((1, 1, 16))
            if l == 1:
                k[..., :8] += junk; v[..., :8] += junk
            o.encode_append(l, [0], 1, k, v)
        outs.append(o.decode_attention(1, [0], g.standard_normal((1, 2, 8))))
    assert np.array_equal(outs[0], outs[1])


# ---------------------------------------------------------------- softmax closed forms
def test_softmax_closed_forms():
    o = small_stack(1, 4, 2, 8, 4, 1, 8, "exact", seed=2)
    fed, g = fill(o, [0], 7)
    q = g.standard_normal((1, 4, 8))
    out, probs = o.decode_attention(0, [0], q, include_current=False, return_probs=True)
    for p in probs:
        assert abs(p.sum() - 1.0) < 1e-14 and p.shape == (7,) and np.all(p > 0)
    # q = 0 -> uniform weights -> mean of the restored values
    out0 = o.decode_attention(0, [0], np.zeros((1, 4, 8)), include_current=False)
    vals = o.restored_rows(0, V, 0)
    for qh in range(4):
        gi = qh // 2
        assert np.max(np.abs(out0[0, qh] - vals[:, gi * 8:(gi + 1) * 8].mean(0))) < 1e-13
    # a single cached token: the output is that token's restored value, whatever q is
    o1 = small_stack(1, 4, 2, 8, 4, 1, 8, "exact", seed=2)
    fill(o1, [0], 1)
    out1 = o1.decode_attention(0, [0], q, include_current=False)
    v1 = o1.restored_rows(0, V, 0)
    for qh in range(4):
        assert np.array_equal(out1[0, qh], v1[0, (qh // 2) * 8:(qh // 2 + 1) * 8])
    # nothing cached, current token only -> exact current value
    o2 = small_stack(1, 4, 2, 8, 4, 1, 8, "exact", seed=2)
    o2.seq_open(0)
    kc = g.standard_normal((1, 1, 16)); vc = g.standard_normal((1, 1, 16))
    o2.encode_append(0, [0], 1, kc, vc)
    out2 = o2.decode_attention(0, [0], q, include_current=True)
    for qh in range(4):
        assert np.array_equal(out2[0, qh], vc[0, 0, (qh // 2) * 8:(qh // 2 + 1) * 8])


def test_scale_is_sqrt_head_dim():
    """Scores must be divided by sqrt(d_k) with d_k the head width (not the model or latent width)."""
    hd = 16
    o = KVCAROracle(1, 1, 1, hd, 4, 1, 4, "exact")
    o.set_reuse_map([-1], [-1])
    o.seq_open(0)
    k = np.zeros((1, 2, hd)); v = np.zeros((1, 2, hd))
    k[0, 0, 0] = 1.0; v[0, 0, 0] = 1.0; v[0, 1, 1] = 1.0
    o.encode_append(0, [0], 2, k, v)
    o.advance([0], 2)
    q = np.zeros((1, 1, hd)); q[0, 0, 0] = 4.0 * math.log(3.0)   # score0 = 4 ln3 / sqrt(16) = ln 3
    out = o.decode_attention(0, [0], q, include_current=False)
    assert abs(out[0, 0, 0] - 0.75) < 1e-14 and abs(out[0, 0, 1] - 0.25) < 1e-14


def test_linear_decoder_identity():
    """With slope 1 the decoder is affine, so q.(W4(BN(W3 z + b3)) + b4) equals a
    dot product of z with an absorbed vector plus a constant (checks decoder +
    score code through different algebra)."""
    o = small_stack(1, 2, 2, 8, 4, 1, 8, "exact", seed=13, slope=1.0)
    fed, g = fill(o, [0], 6)
    q = g.standard_normal((1, 2, 8))
    out, probs = o.decode_attention(0, [0], q, include_current=False, return_probs=True)
    ae = o.ae[(0, K)]
    gam, bet, mu, var = (np.asarray(r, np.float64) for r in ae["dec_bn"])
    sc = gam / np.sqrt(var + ae["bn_eps"])
    rows = [o.locate(0, t)[1] for t in range(6)]
    z = o.pool[(0, K)][rows]
    for qh in range(2):
        w4 = np.asarray(ae["dec_w2"], np.float64)[qh * 8:(qh + 1) * 8]
        b4 = np.asarray(ae["dec_b2"], np.float64)[qh * 8:(qh + 1) * 8]
        u = w4.T @ q[0, qh]                                    # [m]
        absorbed = (np.asarray(ae["dec_w1"], np.float64).T * sc) @ u       # [d]
        const = ((np.asarray(ae["dec_b1"], np.float64) - mu) * sc + bet) @ u + b4 @ q[0, qh]
        s = (z @ absorbed + const) / math.sqrt(8)
        e = np.exp(s - s.max())
        assert np.max(np.abs(e / e.sum() - probs[qh])) < 1e-12


def test_absorbed_last_layer_identity_with_the_nonlinear_decoder():
    """The decoder ends in a bare fully connected layer (Sec. "Network Architecture"), so with the usual LeakyReLU
    slope the score q.k' of a restored key k' = W4_h a + b4_h equals a.(W4_h^T q) + q.b4_h, a being the token's
    activated hidden vector.  The hidden vector is rebuilt here from the cached latents with plain numpy (not the
    oracle's decoder) and the softmax over the absorbed scores must reproduce the oracle's probabilities."""
    o = small_stack(2, 4, 2, 8, 4, 2, 8, "exact", reuse=[(K, 1, 0, 0), (V, 1, 1, 1)], seed=29)
    fed, g = fill(o, [0], 7)
    q = g.standard_normal((1, 4, 8))
    for layer in range(2):
        out, probs = o.decode_attention(layer, [0], q, include_current=False, return_probs=True)
        rows = [o.locate(0, t)[1] for t in range(7)]
        for qh in range(4):
            kvh = qh // 2
            root, head, slot = o.resolve(layer, kvh, K)
            ae = o.ae[(root, K)]
            gam, bet, mu, var = (np.asarray(r, np.float64) for r in ae["dec_bn"])
            pre = o.pool[(root, K)][rows] @ np.asarray(ae["dec_w1"], np.float64).T + np.asarray(ae["dec_b1"], np.float64)
            pre = (pre - mu) / np.sqrt(var + ae["bn_eps"]) * gam + bet
            act = np.where(pre >= 0, pre, ae["leaky_slope"] * pre)                       # [tokens][m]
            w4 = np.asarray(ae["dec_w2"], np.float64)[slot * 8:(slot + 1) * 8]
            b4 = np.asarray(ae["dec_b2"], np.float64)[slot * 8:(slot + 1) * 8]
            s_ = (act @ (w4.T @ q[0, qh]) + b4 @ q[0, qh]) / math.sqrt(8)
            e = np.exp(s_ - s_.max())
            assert np.max(np.abs(e / e.sum() - probs[qh])) < 1e-12, (layer, qh)


# ---------------------------------------------------------------- pages
def test_page_allocation_order_and_locate():
    o = KVCAROracle(1, 1, 1, 8, 4, 4, 6, "exact")
    o.set_reuse_map([-1], [-1])
    for s in (2, 0, 1):
        o.seq_open(s)
    o.reserve([2, 0], 5)                 # two pages each, in call order
    assert o.block_table[2] == [0, 1] and o.block_table[0] == [2, 3]
    o.advance([2, 0], 5)
    assert o.locate(2, 4) == (1, 4) and o.locate(0, 3) == (2, 11) and o.locate(0, 4) == (3, 12)
    o.reserve([2], 3)                    # 5+3 = 8 tokens still fit two pages
    assert o.block_table[2] == [0, 1]
    o.reserve([2], 4)                    # 9 tokens -> third page
    assert o.block_table[2] == [0, 1, 4]
    o.seq_close(0)                       # pages 2,3 released: 3 is handed out next, then 2
    o.reserve([1], 9)
    assert o.block_table[1] == [3, 2, 5]
    with pytest.raises(MemoryError):
        o.reserve([2], 8)
    assert o.block_table[2] == [0, 1, 4]  # nothing taken on failure


def test_physical_page_permutation_does_not_change_outputs():
    def run(scramble):
        o = small_stack(2, 4, 2, 8, 4, 3, 16, "bf16", [(K, 1, 0, 0)], seed=6)
        if scramble:                      # burn and release pages so that the free list is permuted
            o.seq_open(2); o.reserve([2], 11); o.advance([2], 11)
            o.seq_open(1); o.reserve([1], 7); o.seq_close(2); o.seq_close(1)
        g = np.random.default_rng(5)
        o.seq_open(0)
        for l in range(2):
            o.encode_append(l, [0], 13, g.standard_normal((1, 13, 16)), g.standard_normal((1, 13, 16)))
        o.advance([0], 13)
        table = list(o.block_table[0])
        for l in range(2):
            o.encode_append(l, [0], 1, g.standard_normal((1, 1, 16)), g.standard_normal((1, 1, 16)))
        return o.decode_attention(1, [0], g.standard_normal((1, 4, 8))), table
    a, ta = run(False)
    b, tb = run(True)
    assert ta != tb
    assert np.array_equal(a, b)


def test_cached_token_order_is_irrelevant_without_current():
    o = small_stack(1, 2, 2, 8, 4, 2, 16, "exact", seed=3)
    g = np.random.default_rng(9)
    k = g.standard_normal((1, 9, 16)); v = g.standard_normal((1, 9, 16))
    perm = g.permutation(9)
    o.seq_open(0); o.encode_append(0, [0], 9, k, v); o.advance([0], 9)
    o.seq_open(1); o.encode_append(0, [1], 9, k[:, perm], v[:, perm]); o.advance([1], 9)
    q = g.standard_normal((1, 2, 8))
    a = o.decode_attention(0, [0], q, include_current=False)
    b = o.decode_attention(0, [1], q, include_current=False)
    assert np.max(np.abs(a - b)) < 1e-13


# ---------------------------------------------------------------- storage format
def test_bf16_rounding_matches_torch_and_ties_to_even():
    x = np.random.default_rng(0).standard_normal(20000) * np.exp(np.random.default_rng(1).uniform(-20, 20, 20000))
    x32 = x.astype(np.float32)
    ref = torch.tensor(x32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.round_to_bf16(x32.astype(np.float64)), ref)
    # exact ties in fp64: 1 + 2^-8 lies halfway between 1 and 1+2^-7 -> even (1.0); 1+3*2^-8 -> 1+2^-6
    assert orc.round_to_bf16(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert orc.round_to_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    # just above a tie in fp64 (not representable in fp32): must round up, which a detour through fp32 would miss
    assert orc.round_to_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1 + 2.0 ** -7
    assert orc.round_to_bf16(np.array([0.0, -2.5]))[1] == -2.5


def test_storage_mode_rounds_latents_only():
    o = small_stack(1, 2, 2, 8, 4, 1, 8, "bf16", seed=3)
    fed, g = fill(o, [0], 5)
    pool = o.pool[(0, K)]
    rows = [o.locate(0, t)[1] for t in range(5)]
    assert np.array_equal(pool[rows], orc.round_to_bf16(pool[rows]))
    exact = orc.encode(o.ae[(0, K)], fed[(0, 0)][0][0])
    assert np.array_equal(pool[rows], orc.round_to_bf16(exact))
    assert not np.array_equal(pool[rows], exact)


# ---------------------------------------------------------------- Eq. 4
def test_int8_quantisation_eq4():
    x = np.random.default_rng(4).standard_normal(1000) * 3 + 0.7
    q, scale, zp = orc.int8_quantize(x)
    assert q.min() == -128 and q.max() == 127
    assert scale == pytest.approx(255.0 / (x.max() - x.min()))
    assert np.all(q == np.rint(q))
    back = orc.int8_dequantize(q, scale, zp)
    assert np.max(np.abs(back - x)) <= 1.0 / scale + 1e-12     # rounding of x and of the zero point
    # worked by hand: x in {0, 1, 2.55}: scale=100, zp=-128, q = {-128, -28, 127}
    q2, s2, z2 = orc.int8_quantize(np.array([0.0, 1.0, 2.55]))
    assert s2 == pytest.approx(100.0) and z2 == -128 and list(q2) == [-128, -28, 127]
    # the half-way case, worked by hand: x in {0.5, 100, 255.5}: scale = 1, round(0.5) = 0 so zp = -128; the
    # equation gives round(255.5 - 128) = 128 for the maximum, which no int8 holds: the code is 127
    q3, s3, z3 = orc.int8_quantize(np.array([0.5, 100.0, 255.5]))
    assert s3 == 1.0 and z3 == -128 and list(q3) == [-128, -28, 127]
    for seed in range(50):      # codes always fit int8
        r = np.random.default_rng(seed).normal(size=97) * 10 ** np.random.default_rng(seed + 1).uniform(-3, 3)
        qq, _, _ = orc.int8_quantize(r)
        assert qq.min() >= -128 and qq.max() <= 127 and np.all(qq == np.rint(qq))


# ---------------------------------------------------------------- accounting (printed values)
def _records():
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        kind, params, printed, cite = [p.strip() for p in line.split("|")]
        kv = dict(p.split("=") for p in params.split())
        yield kind, kv, printed, cite


def _saving(layers, heads, compressed=0, ratio=1.0, k_heads=0, v_heads=0):
    hd = 64
    o = KVCAROracle(layers, heads, heads, hd, 64, 1, 1, "bf16")
    src = [np.full((layers, heads), -1, int), np.full((layers, heads), -1, int)]
    for which, n in ((K, k_heads), (V, v_heads)):
        if n == "all":
            src[which][1::2, :] = np.arange(heads)           # every second layer reuses the layer below
        else:
            cand = [(l, h) for l in range(1, layers, 2) for h in range(heads)]   # inside compressed layers
            for l, h in cand[:int(n)]:
                src[which][l, h] = h
    o.set_reuse_map(src[K].reshape(-1), src[V].reshape(-1))
    for l in range(int(compressed)):
        for which in (K, V):
            n = len(o.stored_heads(l, which))
            if n:
                i, m, d = synth.ae_dims(n, hd, int(hd * ratio))
                o.ae[(l, which)] = {"in_dim": i, "hidden": m, "latent": d}
    comp, full = o.cache_bytes_per_token()
    return 100.0 * (1.0 - comp / full)


def test_accounting_matches_printed_values():
    seen = 0
    for kind, kv, printed, cite in _records():
        if kind == "eq3_example":
            size = orc.kv_cache_size_bytes(int(kv["bytes"]), int(kv["layers"]), int(kv["d_model"]),
                                           int(kv["seq"]), int(kv["batch"]))
            assert size == 1610612736
            assert abs(size / 1e9 - 1.61) < 0.005, cite
        elif kind == "eq3_ratio":
            assert abs(1610612736 / float(kv["model_bytes"]) - float(printed)) < 0.005, cite
        else:
            args = dict(layers=int(kv["layers"]), heads=int(kv["heads"]))
            if "compressed" in kv:
                args.update(compressed=int(kv["compressed"]), ratio=float(kv["ratio"]))
            for n in ("k_heads", "v_heads"):
                if n in kv:
                    args[n] = kv[n] if kv[n] == "all" else int(kv[n])
            assert abs(_saving(**args) - float(printed)) < 0.1, (cite, _saving(**args))
        seen += 1
    assert seen == 14


def test_bytes_per_token_of_the_benchmark_shapes():
    # GPT-2-small shape, 2x autoencoder everywhere, no reuse: 12 layers * 2 * 384 * 2 B
    for name, expect_c, expect_f in (("c2", 12 * 2 * 384 * 2, 12 * 2 * 768 * 2), ("c3", 22 * 2 * 128 * 2, 22 * 2 * 256 * 2)):
        w = synth.CONFIGS[name]
        o = KVCAROracle(w.n_layers, w.n_q_heads, w.n_kv_heads, 64, 64, 1, 1, "bf16")
        o.set_reuse_map([-1] * (w.n_layers * w.n_kv_heads), [-1] * (w.n_layers * w.n_kv_heads))
        for l in range(w.n_layers):
            for which in (K, V):
                i, m, d = synth.ae_dims(w.n_kv_heads, 64, w.latent_per_head)
                o.ae[(l, which)] = {"in_dim": i, "hidden": m, "latent": d}
        assert o.cache_bytes_per_token() == (expect_c, expect_f)


# ---------------------------------------------------------------- generator sanity (not method arithmetic)
def test_reuse_map_generator_counts():
    for name, n in (("c2", 33), ("c3", 17)):
        w = synth.CONFIGS[name]
        src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
        assert int((src >= 0).sum()) == n
        assert np.all(src[:w.n_kv_heads] == -1)
        again = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
        assert np.array_equal(src, again)


# ---------------------------------------------------------------- Alg. 2: head distances and the reuse choice
def test_head_l1_distance_closed_forms_and_brute_force():
    """Alg. 2's distance step (an L1 norm between the same head in two adjacent layers), pinned by cases with a known answer:
    equal layers -> 0; a per-head constant offset -> its magnitude; loops written out on a tiny case (which
    catches a wrong layer pairing, a wrong head slice or a wrong divisor); scaling; row order."""
    rng = np.random.default_rng(5)
    L, R, H, hd = 4, 7, 3, 4
    base = rng.normal(size=(R, H * hd))
    # (1) identical layers
    x = np.stack([base] * L)
    assert np.array_equal(orc.head_l1_distance(x, H), np.zeros((L - 1, H)))
    # (2) layer l = layer l-1 + delta[l][h] on every channel of head h: distance = |delta|
    delta = rng.normal(size=(L, H))
    x = np.zeros((L, R, H * hd))
    x[0] = base
    for l in range(1, L):
        x[l] = x[l - 1] + np.repeat(delta[l], hd)[None, :]
    np.testing.assert_allclose(orc.head_l1_distance(x, H), np.abs(delta[1:]), rtol=0, atol=1e-12)
    # (3) brute force, every index written out
    x = rng.normal(size=(L, R, H * hd))
    want = np.zeros((L - 1, H))
    for l in range(1, L):
        for h in range(H):
            tot = 0.0
            for r in range(R):
                for c in range(hd):
                    tot += abs(x[l][r][h * hd + c] - x[l - 1][r][h * hd + c])
            want[l - 1][h] = tot / (R * hd)
    got = orc.head_l1_distance(x, H)
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=0)
    assert not np.allclose(got, orc.head_l1_distance(x[::-1], H)[::-1][:, ::-1])    # heads are not interchangeable
    # (4) |a| D(x) = D(a x); the order of the rows is irrelevant; a constant added to every layer cancels
    np.testing.assert_allclose(orc.head_l1_distance(-2.5 * x, H), 2.5 * got, rtol=1e-13)
    np.testing.assert_allclose(orc.head_l1_distance(x[:, rng.permutation(R)], H), got, rtol=1e-13)
    np.testing.assert_allclose(orc.head_l1_distance(x + 3.0, H), got, rtol=1e-12)
    # (5) mini-batches of equal size average to the distance of their union (the text averages over mini-batches)
    a, b = rng.normal(size=(L, R, H * hd)), rng.normal(size=(L, R, H * hd))
    both = np.concatenate([a, b], axis=1)
    np.testing.assert_allclose(0.5 * (orc.head_l1_distance(a, H) + orc.head_l1_distance(b, H)),
                               orc.head_l1_distance(both, H), rtol=1e-13)


def test_reuse_map_from_l1_picks_the_closest_heads():
    """Alg. 2: heads whose distance to the layer below is smallest reuse it.  Hand-made distances with a known
    ranking (including a tie) and the table format the cache expects (layer 0 never reuses; entry = same head)."""
    dist = np.array([[0.9, 0.1, 0.5],       # layer 1 vs 0
                     [0.1, 0.7, 0.3],       # layer 2 vs 1   (0.1 ties with layer 1, head 1: the lower layer wins)
                     [0.2, 0.8, 0.6]])      # layer 3 vs 2
    none = orc.reuse_map_from_l1(dist, 0)
    assert none.dtype == np.int32 and none.tolist() == [-1] * 12
    one = orc.reuse_map_from_l1(dist, 1)
    assert one.tolist() == [-1, -1, -1, -1, 1, -1, -1, -1, -1, -1, -1, -1]
    four = orc.reuse_map_from_l1(dist, 4)
    # ranking: (1,1)=0.1, (2,0)=0.1, (3,0)=0.2, (2,2)=0.3
    assert four.tolist() == [-1, -1, -1, -1, 1, -1, 0, -1, 2, 0, -1, -1]
    assert orc.reuse_map_from_l1(dist, 9).tolist() == [-1, -1, -1, 0, 1, 2, 0, 1, 2, 0, 1, 2]
    # the table is accepted by the cache model and resolves through chains (layer 3 head 0 -> layer 1 head 0)
    o = KVCAROracle(4, 3, 3, 4, page_tokens=2, max_seqs=1, max_pages=4, storage="exact")
    o.set_reuse_map(four, four)
    assert o.resolve(3, 0, K)[:2] == (1, 0)


def test_int8_latent_rows_stay_within_half_a_step():
    """Eq. 4 per cached row (the storage mode an int8 latent cache would have): every value comes back within
    half a quantisation step of itself, the row's extremes within one step, a constant row unchanged, and the
    cache accounting charges one byte per element plus the row's scale and zero-point."""
    rng = np.random.default_rng(9)
    z = rng.normal(size=(5, 7, 48)) * rng.uniform(0.1, 10.0, size=(5, 7, 1))
    z[2, 3] = 1.25                                              # a row of equal values
    back = orc.int8_rows(z)
    step = (z.max(axis=-1, keepdims=True) - z.min(axis=-1, keepdims=True)) / 255.0
    assert np.all(np.abs(back - z) <= 0.5 * step + 1e-12)
    assert np.array_equal(back[2, 3], z[2, 3])
    row = z[0, 0]
    q, scale, zp = orc.int8_quantize(row)
    assert q.min() >= -128 and q.max() <= 127 and np.all(q == np.rint(q))
    assert abs(orc.int8_dequantize(q, scale, zp).max() - row.max()) <= step[0, 0, 0]
    # rows are independent: quantising a row alone or inside a batch gives the same values
    assert np.array_equal(orc.int8_rows(z[1, 2][None])[0], back[1, 2])
    # the cache model stores them and accounts for them
    o = KVCAROracle(2, 2, 2, 4, page_tokens=2, max_seqs=1, max_pages=4, storage="int8")
    o.set_reuse_map([-1, -1, 0, -1], [-1, -1, -1, -1])          # layer 1 K head 0 reuses layer 0
    comp, full = o.cache_bytes_per_token()
    assert comp == (8 + 8 + 4 + 8) * 1 + 4 * 8                  # widths 8, 8, 4, 8 at one byte + four rows' parameters
    assert full == 2 * 2 * 8 * 2                                # against 16-bit raw K/V
    o.seq_open(0)
    k = rng.normal(size=(1, 3, 8)); v = rng.normal(size=(1, 3, 8))
    o.encode_append(0, [0], 3, k, v)
    stored = o._pool(0, K)[[o.locate(0, t)[1] for t in range(3)]]
    np.testing.assert_array_equal(stored, orc.int8_rows(k[0]))
