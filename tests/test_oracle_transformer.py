"""Pins for the transformer-layer oracle and the layer-wise caching loop (CPU only)."""
import math

import numpy as np
import torch

from oracle import llmcache_oracle as O
from oracle import transformer_oracle as T


def rng(seed):
    return np.random.Generator(np.random.Philox(key=seed))


def bf16_bits(x):
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def make_weights(r, d, ffn, scale=0.05):
    g = lambda *s: bf16_bits(r.standard_normal(s) * scale)
    f = lambda *s: (r.standard_normal(s) * 0.1).astype(np.float32)
    return T.LayerWeights(w_qkv=g(3 * d, d), b_qkv=f(3 * d), w_o=g(d, d), b_o=f(d),
                          ln1_g=(1 + f(d)).astype(np.float32), ln1_b=f(d), w_1=g(ffn, d), b_1=f(ffn),
                          w_2=g(d, ffn), b_2=f(d), ln2_g=(1 + f(d)).astype(np.float32), ln2_b=f(d))


def torch_layer(w, d, heads, ffn, pre_ln, tanh_gelu):
    act = (lambda x: torch.nn.functional.gelu(x, approximate="tanh")) if tanh_gelu else torch.nn.functional.gelu
    m = torch.nn.TransformerEncoderLayer(d, heads, ffn, dropout=0.0, activation=act, batch_first=True,
                                         norm_first=pre_ln, dtype=torch.float64)
    W = lambda b: torch.from_numpy(O.bf16_to_f32(b).astype(np.float64))
    V = lambda v: torch.from_numpy(np.asarray(v, np.float32).astype(np.float64))
    with torch.no_grad():
        m.self_attn.in_proj_weight.copy_(W(w.w_qkv)); m.self_attn.in_proj_bias.copy_(V(w.b_qkv))
        m.self_attn.out_proj.weight.copy_(W(w.w_o)); m.self_attn.out_proj.bias.copy_(V(w.b_o))
        m.linear1.weight.copy_(W(w.w_1)); m.linear1.bias.copy_(V(w.b_1))
        m.linear2.weight.copy_(W(w.w_2)); m.linear2.bias.copy_(V(w.b_2))
        m.norm1.weight.copy_(V(w.ln1_g)); m.norm1.bias.copy_(V(w.ln1_b))
        m.norm2.weight.copy_(V(w.ln2_g)); m.norm2.bias.copy_(V(w.ln2_b))
    return m.eval()


def test_layer_matches_torch_reference_layer_both_arrangements():
    r = rng(1)
    n, d, heads, ffn = 12, 32, 4, 64
    w = make_weights(r, d, ffn)
    x = bf16_bits(r.standard_normal((n, d)))
    xt = torch.from_numpy(O.bf16_to_f32(x).astype(np.float64))[None]
    for pre_ln, causal, tanh_gelu in ((False, False, False), (True, True, True)):
        m = torch_layer(w, d, heads, ffn, pre_ln, tanh_gelu)
        mask = torch.triu(torch.full((n, n), float("-inf"), dtype=torch.float64), diagonal=1) if causal else None
        with torch.no_grad():
            ref = m(xt, src_mask=mask)[0].numpy()
        exact = T.layer_forward_f64(x, w, heads, pre_ln, causal, tanh_gelu)
        assert np.max(np.abs(exact - ref)) < 1e-10
        got = T.layer_forward(x, w, heads, pre_ln, causal, tanh_gelu)
        assert np.array_equal(got, bf16_bits(exact))


def test_layer_norm_and_gelu_against_library():
    r = rng(2)
    x = r.standard_normal((5, 16))
    g = r.standard_normal(16); b = r.standard_normal(16)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (16,), torch.from_numpy(g), torch.from_numpy(b)).numpy()
    assert np.allclose(T.layer_norm(x, g, b), ref, atol=1e-12)
    assert np.allclose(T.gelu_erf(x), torch.nn.functional.gelu(torch.from_numpy(x)).numpy(), atol=1e-14)
    assert np.allclose(T.gelu_tanh(x), torch.nn.functional.gelu(torch.from_numpy(x), approximate="tanh").numpy(), atol=1e-14)
    assert abs(T.gelu_erf(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15      # x * Phi(x) at x = 1


def test_attention_hand_worked_and_causal_mask():
    # one head, dh = 1: scores q_i * k_j; softmax rows worked by hand
    qkv = np.array([[1.0, 0.0, 2.0], [1.0, math.log(3.0), 4.0]])                 # columns q | k | v
    out = T.attention(qkv, heads=1, causal=False)
    assert np.allclose(out[:, 0], [2.0 * 0.25 + 4.0 * 0.75] * 2)                 # softmax([0, ln 3]) = [1/4, 3/4]
    out = T.attention(qkv, heads=1, causal=True)
    assert np.allclose(out[:, 0], [2.0, 3.5])                                    # row 0 sees only itself
    r = rng(3)
    qkv = r.standard_normal((9, 3 * 8))
    base = T.attention(qkv, heads=2, causal=True)
    qkv2 = qkv.copy(); qkv2[6:] += 1.0                                           # change the future
    assert np.array_equal(T.attention(qkv2, heads=2, causal=True)[:6], base[:6])
    perm = r.permutation(9)                                                      # bidirectional: equivariant
    assert np.allclose(T.attention(qkv[perm], 2, False), T.attention(qkv, 2, False)[perm], atol=1e-12)


def test_rounded_intermediates_stay_close_to_exact():
    r = rng(4)
    n, d, heads, ffn = 16, 64, 4, 128
    w = make_weights(r, d, ffn)
    x = bf16_bits(r.standard_normal((n, d)))
    a = O.bf16_to_f32(T.layer_forward(x, w, heads)).astype(np.float64)
    b = O.bf16_to_f32(T.layer_forward(x, w, heads, round_bf16=True)).astype(np.float64)
    assert np.sqrt(np.mean((a - b) ** 2)) / np.sqrt(np.mean(a ** 2)) < 2e-2
    assert not np.array_equal(a, b)


def test_infer_chain_property_of_the_caching_loop():
    r = rng(5)
    B, n, d, heads, ffn, Lyr = 4, 8, 64, 4, 128, 3
    layers = [make_weights(r, d, ffn) for _ in range(Lyr)]
    banks = [O.Bank(capacity=16, seq_len=n, d_model=d, fp_dim=d, tau=0.9) for _ in range(Lyr)]
    h0 = bf16_bits(r.standard_normal((B, n, d)))
    out1, hits1 = T.infer(banks, layers, h0, heads)
    assert hits1 == [0, 0, 0]
    for b in range(B):                                  # all misses: the plain forward pass
        h = h0[b]
        for w in layers:
            h = T.layer_forward(h, w, heads)
        assert np.array_equal(out1[b], h.reshape(-1))
    # the same batch again: served from the banks at every layer, bit-identical output (Algorithm 1)
    out2, hits2 = T.infer(banks, layers, h0, heads)
    assert hits2 == [B, B, B] and np.array_equal(out1, out2)
    # a near-duplicate of sequence 0 hits at layer 1 and therefore at every deeper layer, with sequence 0's output
    near = h0.copy()
    near[1] = bf16_bits(O.bf16_to_f32(h0[0]) + 0.02 * r.standard_normal((n, d)).astype(np.float32))
    out3, hits3 = T.infer(banks, layers, near, heads)
    assert hits3 == [B, B, B] and np.array_equal(out3[1], out1[0])


def test_divergence_monitor_flags_only_entries_whose_stored_output_drifted():
    r = rng(6)
    B, n, d, heads, ffn = 6, 8, 64, 4, 128
    w = make_weights(r, d, ffn)
    bank = O.Bank(capacity=16, seq_len=n, d_model=d, fp_dim=d, tau=0.9)
    h = bf16_bits(r.standard_normal((B, n, d)))
    outs = np.stack([T.layer_forward(h[b], w, heads).reshape(-1) for b in range(B)])
    O.commit(bank, O.probe(bank, h, "bf16"), outs)
    # corrupt the stored output of slot 2 (a stale entry: the layer no longer produces it)
    bank.act[2] = bf16_bits(O.bf16_to_f32(bank.act[2]) * 1.5)
    pr = O.probe(bank, h, "bf16")
    assert pr.hit.sum() == B
    checked, dropped = T.divergence_check(bank, w, h, pr, heads, stride=1, bound=0.05)
    rels = {slot: rel for _, slot, rel in checked}
    assert dropped == 1 and bank.valid[2] == 0 and bank.valid.sum() == B - 1
    assert abs(rels[2] - 0.5) < 0.01 and all(rel == 0.0 for s, rel in rels.items() if s != 2)
    # sampling: every third hit only
    pr = O.probe(bank, h, "bf16")
    checked, dropped = T.divergence_check(bank, w, h, pr, heads, stride=3, bound=0.05)
    assert [b for b, _, _ in checked] == [int(pr.hit_idx[i]) for i in range(0, len(pr.hit_idx), 3)] and dropped == 0


def test_embed_hand_worked_library_and_degenerate_cases():
    """h_0 = E(X) of Algorithm 1.  (a) one row by hand: [1, 3] has mean 2 and variance 1, so with eps = 0 the
    normalised row is [-1, 1], and with gain [2, 1], bias [0.5, 0] it is [-1.5, 1]; (b) the library's
    embedding lookup + layer_norm in float64; (c) a token table of zeros leaves the position rows, row i at
    position i (an index mix-up between position and sequence would show); (d) an id outside the table gives a
    zero row; (e) the stored form is the bf16 rounding of the exact one."""
    f2b = lambda a: O.bf16_round(np.asarray(a, dtype=np.float32))
    E = f2b([[1.0, 3.0], [2.0, 2.0]])
    P0 = f2b([[0.0, 0.0]])
    got = T.embed_f64(np.array([[0]]), E, P0, True, None, None, 0.0)
    assert np.allclose(got, [[[-1.0, 1.0]]], atol=1e-15)
    got = T.embed_f64(np.array([[0]]), E, P0, True, np.float32([2, 1]), np.float32([0.5, 0]), 0.0)
    assert np.allclose(got, [[[-1.5, 1.0]]], atol=1e-15)
    assert np.array_equal(T.embed_f64(np.array([[1]]), E, f2b([[0.5, -0.25]]), False), [[[2.5, 1.75]]])

    rng = np.random.default_rng(3)
    vocab, n, d, S = 50, 7, 24, 5
    Eb, Pb = f2b(rng.standard_normal((vocab, d))), f2b(rng.standard_normal((n, d)))
    g, b = rng.standard_normal(d).astype(np.float32), rng.standard_normal(d).astype(np.float32)
    tok = rng.integers(0, vocab, (S, n))
    te = torch.from_numpy(O.bf16_to_f32(Eb).astype(np.float64))
    tp = torch.from_numpy(O.bf16_to_f32(Pb).astype(np.float64))
    x = torch.nn.functional.embedding(torch.from_numpy(tok), te) + tp[None]
    ref = torch.nn.functional.layer_norm(x, (d,), torch.from_numpy(g.astype(np.float64)),
                                         torch.from_numpy(b.astype(np.float64)), 1e-5).numpy()
    got = T.embed_f64(tok, Eb, Pb, True, g, b, 1e-5)
    assert np.abs(got - ref).max() < 1e-12
    assert np.abs(T.embed_f64(tok, Eb, Pb, False) - x.numpy()).max() == 0.0
    assert np.abs(T.embed_f64(tok, Eb, None, False) - te.numpy()[tok]).max() == 0.0

    zeros = np.zeros((vocab, d), dtype=np.uint16)
    got = T.embed_f64(tok, zeros, Pb, False)
    for s in range(S):
        assert np.array_equal(got[s], O.bf16_to_f32(Pb).astype(np.float64))

    bad = tok.copy()
    bad[2, 3], bad[4, 0] = vocab, -1
    got = T.embed_f64(bad, Eb, Pb, True, g, b, 1e-5)
    assert not got[2, 3].any() and not got[4, 0].any() and got[2, 2].any()

    bits = T.embed(tok, Eb, Pb, True, g, b, 1e-5)
    assert bits.dtype == np.uint16 and np.array_equal(bits, O.bf16_round(ref.astype(np.float32)))
