"""Miss-path transformer layer and the layer-wise caching loop (Algorithm 1) against the oracle.

Tolerance (derived): the CUDA layer keeps seven intermediate tensors in bf16 and accumulates in fp32.
Against the oracle that rounds at the same storage points the remaining differences are fp32 vs float64
accumulation, the fast exponential, and the occasional bf16 rounding that falls the other way (one step =
2^-8 relative on that element), and the bf16 rounding of the attention probabilities that feed the
tensor-core P V product (about 1e-3 relative each, which the oracle does not have):
root-mean-square error <= 6e-3 of the output's RMS (1.5 bf16 steps) and no element further
than 4 bf16 steps of the element + 2 % of the output's RMS (an element near zero inherits the rounding
steps of the larger terms it is the sum of).  Against the oracle that rounds nothing: RMS error <= 2e-2."""
import numpy as np
import pytest
import torch

from oracle import llmcache_oracle as O
from oracle import transformer_oracle as T
from paper_2512_16843_b200 import binding as L
from paper_2512_16843_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def oracle_weights(w):
    conv = lambda t: synth.bf16_bits(t) if t.dtype == torch.bfloat16 else t.cpu().numpy()
    return T.LayerWeights(**{k: conv(w[k]) for k in L.WEIGHT_NAMES})


def rel_rms(a, b):
    return float(np.sqrt(np.mean((a - b) ** 2)) / np.sqrt(np.mean(b ** 2)))


def check_layer_output(got_bits, x_bits, ow, heads, **kw):
    got = O.bf16_to_f32(got_bits).astype(np.float64)
    ref_r = O.bf16_to_f32(T.layer_forward(x_bits, ow, heads, round_bf16=True, **kw)).astype(np.float64)
    ref_e = T.layer_forward_f64(x_bits, ow, heads, **kw)
    assert rel_rms(got, ref_r) <= 6e-3, rel_rms(got, ref_r)
    assert np.all(np.abs(got - ref_r) <= 4 * 2.0 ** -8 * np.abs(ref_r) + 0.02 * np.sqrt(np.mean(ref_r ** 2)))
    assert rel_rms(got, ref_e) <= 2e-2, rel_rms(got, ref_e)


@pytest.mark.parametrize("n,d,heads,ffn,S,pre_ln,causal,tanh", [
    (40, 128, 2, 256, 3, False, False, False),       # ragged everywhere
    (130, 192, 3, 320, 2, True, True, True),         # two query tiles, causal, odd tile counts
    (128, 768, 12, 3072, 2, False, False, False),    # BERT-base layer
    (256, 768, 12, 3072, 1, True, True, True),       # GPT-2-small layer
    (200, 1024, 16, 4096, 3, False, False, False),   # BERT-large layer; 600 rows: four full row blocks and a partial one
])
def test_layer_forward_matches_oracle(n, d, heads, ffn, S, pre_ln, causal, tanh):
    w = synth.layer_weights(d, ffn, 100 + d + n, DEV)
    # larger weights than the 0.02 initialisation so that every sub-block matters in the output
    for k in ("w_qkv", "w_o", "w_1", "w_2"):
        w[k] = (w[k].float() * 3.0).to(torch.bfloat16)
    layer = L.Layer(w, heads=heads, seq_len=n, max_seqs=S, pre_ln=pre_ln, causal=causal, tanh_gelu=tanh)
    x = synth.randn((S, n, d), 7, DEV, torch.bfloat16)
    out = torch.zeros_like(x)
    layer.forward(x, out)
    torch.cuda.synchronize()
    assert layer.status() == L.OK
    ow = oracle_weights(w)
    for s in range(S):
        check_layer_output(synth.bf16_bits(out[s]), synth.bf16_bits(x[s]), ow, heads,
                           pre_ln=pre_ln, causal=causal, tanh_gelu=tanh)
    layer.close()


def test_layer_forward_with_device_side_count():
    n, d, heads, ffn, S = 64, 128, 2, 256, 5
    w = synth.layer_weights(d, ffn, 31, DEV)
    layer = L.Layer(w, heads=heads, seq_len=n, max_seqs=S)
    x = synth.randn((S, n, d), 8, DEV, torch.bfloat16)
    full = torch.zeros_like(x)
    layer.forward(x, full)
    for count in (0, 2, 5, 9):
        out = torch.full_like(x, 7.0)
        cnt = torch.tensor([count], dtype=torch.int32, device=DEV)
        layer.forward(x, out, n_seqs_dev=cnt)
        torch.cuda.synchronize()
        m = min(count, S)
        assert torch.equal(out[:m].view(torch.int16), full[:m].view(torch.int16))     # same bits as the full run
        assert torch.all(out[m:] == 7.0)                                             # nothing beyond the count
    with pytest.raises(L.LLMCacheError) as e:
        layer.forward(torch.zeros((S + 1, n, d), dtype=torch.bfloat16, device=DEV), torch.zeros((S + 1, n, d), dtype=torch.bfloat16, device=DEV))
    assert e.value.status == L.ERR_SHAPE
    layer.close()


@pytest.mark.parametrize("pre_ln", [False, True])
def test_infer_algorithm1_matches_oracle_and_chain_property(pre_ln):
    n, d, heads, ffn, B, Lyr, N, k = 48, 128, 2, 256, 12, 3, 64, 64
    ws = [synth.layer_weights(d, ffn, 200 + 20 * l, DEV) for l in range(Lyr)]
    for w in ws:
        for key in ("w_qkv", "w_o", "w_1", "w_2"):
            w[key] = (w[key].float() * 3.0).to(torch.bfloat16)
    proj = synth.projection(d, k, 9, DEV)
    kw = dict(pre_ln=pre_ln, causal=pre_ln, tanh_gelu=pre_ln)
    layers = [L.Layer(w, heads=heads, seq_len=n, max_seqs=B, **kw) for w in ws]
    banks = [L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, proj=proj, tau=0.9) for _ in range(Lyr)]
    obanks = [O.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, tau=0.9, proj=synth.bf16_bits(proj)) for _ in range(Lyr)]
    ows = [oracle_weights(w) for w in ws]
    bufs = L.ProbeBuffers(B, k, DEV)
    mk = lambda: torch.zeros((B, n, d), dtype=torch.bfloat16, device=DEV)
    buf_a, buf_b, h_miss, miss_out = mk(), mk(), mk(), mk()
    handles_b, handles_l = [b.handle for b in banks], [l.handle for l in layers]

    def run(h0, use_banks=True):
        ptr = L.llmcache_infer(handles_b if use_banks else None, handles_l, h0, B, None, buf_a, buf_b, h_miss, miss_out, bufs.io)
        torch.cuda.synchronize()
        return (buf_a if ptr == buf_a.data_ptr() else buf_b).clone()

    h0 = synth.randn((B, n, d), 3, DEV, torch.bfloat16)
    plain = run(h0, use_banks=False)                     # no caching: every layer in full
    out1 = run(h0)                                       # empty banks: all miss, same computation
    assert torch.equal(plain.view(torch.int16), out1.view(torch.int16))
    ref1, hits1 = T.infer(obanks, ows, synth.bf16_bits(h0), heads, round_bf16=True, **kw)
    assert hits1 == [0] * Lyr and [b.stats()["hits"] for b in banks] == [0] * Lyr
    got = O.bf16_to_f32(synth.bf16_bits(out1)).astype(np.float64)
    ref = O.bf16_to_f32(ref1).astype(np.float64).reshape(got.shape)
    assert rel_rms(got, ref) <= 1e-2
    # same batch again: every layer is served from its bank; the output has the same bits (Algorithm 1)
    out2 = run(h0)
    assert [b.stats()["hits"] for b in banks] == [B] * Lyr
    assert torch.equal(out1.view(torch.int16), out2.view(torch.int16))
    ref2, hits2 = T.infer(obanks, ows, synth.bf16_bits(h0), heads, round_bf16=True, **kw)
    assert hits2 == [B] * Lyr
    # a mixed batch: near-duplicates hit at layer 1 and hence at every deeper layer with the donor's output
    mixed = h0.clone()
    mixed[1] = (h0[0].float() + 0.02 * synth.randn((n, d), 4, DEV)).to(torch.bfloat16)
    mixed[5:9] = synth.randn((4, n, d), 5, DEV, torch.bfloat16)
    out3 = run(mixed)
    ref3, hits3 = T.infer(obanks, ows, synth.bf16_bits(mixed), heads, round_bf16=True, **kw)
    gpu_hits = [b.stats()["hits"] - B for b in banks]
    assert gpu_hits == hits3 == [B - 4] * Lyr
    assert torch.equal(out3[1].view(torch.int16), out1[0].view(torch.int16))
    assert all(l.status() == L.OK for l in layers) and all(b.status() == L.OK for b in banks)
    for o in layers + banks:
        o.close()


def test_infer_with_fingerprint_on_write_equals_plain_loop():
    """Same batches through llmcache_infer and llmcache_infer_pooled (own banks each): same hits per layer,
    same output bits.  (The two differ only in where the position means of h_1..h_{L-1} are taken.)  A third
    set of banks, created with fused_pool, goes through llmcache_infer, which must take the pooled path by
    itself: same bits again, and the same number of kernel launches as the explicit pooled loop."""
    n, d, heads, ffn, B, Lyr, N, k = 40, 128, 2, 256, 14, 4, 64, 64
    ws = [synth.layer_weights(d, ffn, 400 + 20 * l, DEV) for l in range(Lyr)]
    for w in ws:
        for key in ("w_qkv", "w_o", "w_1", "w_2"):
            w[key] = (w[key].float() * 3.0).to(torch.bfloat16)
    proj = synth.projection(d, k, 19, DEV)
    layers = [L.Layer(w, heads=heads, seq_len=n, max_seqs=B) for w in ws]
    mkb = lambda fused: [L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, proj=proj, tau=0.9,
                                fused_pool=fused) for _ in range(Lyr)]
    banks_a, banks_b, banks_c = mkb(0), mkb(1), mkb(1)
    bufs = L.ProbeBuffers(B, k, DEV)
    mk = lambda: torch.zeros((B, n, d), dtype=torch.bfloat16, device=DEV)
    buf_a, buf_b, h_miss, miss_out = mk(), mk(), mk(), mk()
    pooled = torch.zeros((B, d), dtype=torch.float32, device=DEV)
    hl = [l.handle for l in layers]

    def run(h0, fused):
        if fused == 2:
            ptr = L.llmcache_infer([b.handle for b in banks_c], hl, h0, B, None, buf_a, buf_b, h_miss, miss_out, bufs.io)
        elif fused:
            ptr = L.llmcache_infer_pooled([b.handle for b in banks_b], hl, h0, B, None, buf_a, buf_b, h_miss, miss_out,
                                          bufs.io, pooled)
        else:
            ptr = L.llmcache_infer([b.handle for b in banks_a], hl, h0, B, None, buf_a, buf_b, h_miss, miss_out, bufs.io)
        torch.cuda.synchronize()
        return (buf_a if ptr == buf_a.data_ptr() else buf_b).clone()

    h0 = synth.randn((B, n, d), 3, DEV, torch.bfloat16)
    batches = [h0]
    mixed = h0.clone()
    mixed[1] = (h0[0].float() + 0.02 * synth.randn((n, d), 4, DEV)).to(torch.bfloat16)
    mixed[5:9] = synth.randn((4, n, d), 5, DEV, torch.bfloat16)
    batches += [h0, mixed, synth.randn((B, n, d), 6, DEV, torch.bfloat16), mixed]
    prev_a, prev_b = [0] * Lyr, [0] * Lyr
    total = 0
    for i, hb in enumerate(batches):
        oa, ob, oc = run(hb, False), run(hb, True), run(hb, 2)
        assert torch.equal(oc.view(torch.int16), ob.view(torch.int16)), f"batch {i} (banks with fused_pool through llmcache_infer)"
        ha = [b.stats()["hits"] for b in banks_a]
        hb_ = [b.stats()["hits"] for b in banks_b]
        assert [x - y for x, y in zip(ha, prev_a)] == [x - y for x, y in zip(hb_, prev_b)], f"batch {i}"
        total += ha[0] - prev_a[0]
        prev_a, prev_b = ha, hb_
        assert torch.equal(oa.view(torch.int16), ob.view(torch.int16)), f"batch {i}"
    assert total >= B + (B - 4)
    launches_a = sum(b.stats()["kernel_launches"] for b in banks_a)
    launches_b = sum(b.stats()["kernel_launches"] for b in banks_b)
    assert launches_b != launches_a                      # the pooled loop really took the other path
    assert sum(b.stats()["kernel_launches"] for b in banks_c) == launches_b
    assert [b.stats()["hits"] for b in banks_c] == [b.stats()["hits"] for b in banks_b]
    assert all(l.status() == L.OK for l in layers) and all(b.status() == L.OK for b in banks_a + banks_b + banks_c)
    for o in layers + banks_a + banks_b + banks_c:
        o.close()


def test_divergence_monitor_matches_oracle():
    """Stored outputs that no longer match what the layer produces are found and invalidated; the relative
    differences agree with the oracle's within the layer tolerance (absolute 1e-2 on a quantity of order
    0..1), decisions within that distance of the bound would be reported, not failed (none here)."""
    n, d, heads, ffn, B, N, k, stride = 32, 128, 2, 256, 20, 64, 128, 3
    w = synth.layer_weights(d, ffn, 77, DEV)
    for key in ("w_qkv", "w_o", "w_1", "w_2"):
        w[key] = (w[key].float() * 3.0).to(torch.bfloat16)
    layer = L.Layer(w, heads=heads, seq_len=n, max_seqs=B)
    bank = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, tau=0.9)
    bufs = L.ProbeBuffers(B, k, DEV)
    h = synth.randn((B, n, d), 5, DEV, torch.bfloat16)
    h_out = torch.zeros((B, n * d), dtype=torch.bfloat16, device=DEV)
    outs = torch.zeros((B, n, d), dtype=torch.bfloat16, device=DEV)
    layer.forward(h, outs)
    bank.probe(h, bufs, h_out=h_out)
    bank.commit(outs, bufs, h_out=h_out)
    torch.cuda.synchronize()
    # make three stored outputs stale (slots 0, 6 and 7 are the entries of sequences 0, 6, 7)
    act = bank.export(L.WHAT_ACT)
    for s_, f in ((0, 1.3), (6, 0.5), (7, 1.02)):
        act[s_] = (act[s_].float() * f).to(torch.bfloat16)
    bank.import_(L.WHAT_ACT, act)
    bank.probe(h, bufs, h_out=h_out)
    bank.commit(outs, bufs, h_out=h_out)              # all hits: nothing to insert
    torch.cuda.synchronize()
    assert int(bufs.counts[0]) == B
    S = (B + stride - 1) // stride
    h_sample = torch.zeros((S, n, d), dtype=torch.bfloat16, device=DEV)
    out_sample = torch.zeros_like(h_sample)
    rel = torch.zeros(S, dtype=torch.float32, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int32, device=DEV)
    from tests import parity_util as U
    ob = U.oracle_bank_like(bank)
    U.pull_state(bank, ob)
    pr = U.gpu_probe_result(bufs, B, ob.tick)
    L.llmcache_divergence_check(bank.handle, layer.handle, h, bufs.io, stride, 0.1, h_sample, out_sample, rel, cnt)
    torch.cuda.synchronize()
    checked, dropped = T.divergence_check(ob, oracle_weights(w), synth.bf16_bits(h), pr, heads, stride, 0.1,
                                          round_bf16=True)
    assert cnt.tolist() == [len(checked), dropped] and dropped == 2        # samples 0, 3, 6, ...: slots 0 and 6
    got = rel.cpu().numpy()
    for i, (_, slot, r) in enumerate(checked):
        assert abs(got[i] - r) <= 1e-2, (i, slot, got[i], r)
    assert np.array_equal(bank.export(L.WHAT_VALID).numpy(), ob.valid)
    assert bank.status() == L.OK and layer.status() == L.OK
    layer.close(); bank.close()


@pytest.mark.parametrize("S,n,d,vocab,ln,affine,pos", [
    (3, 40, 128, 1000, True, True, True),          # ragged: 4 chunks of a lane's 4 hold data on half the lanes
    (2, 128, 768, 30522, True, False, True),       # BERT-base embeddings (the workload generator's recipe)
    (2, 64, 768, 50257, False, False, True),       # GPT-2-style: no layer norm
    (1, 33, 1024, 777, True, True, False),         # no position term
    (2, 17, 2048, 512, True, True, True),          # eight chunks per lane
    (1, 9, 4096, 64, True, True, True),            # any width: the sum is formed three times
])
def test_embed_matches_oracle(S, n, d, vocab, ln, affine, pos):
    """h_0 = E(X): every element within one bf16 step of the float64 oracle (the sum of two bf16 numbers is exact
    in fp32; the layer norm's fp32 mean and variance differ from float64 by ~1e-7 relative, which can flip a
    rounding), and at most 1 % of them different at all."""
    E = synth.randn((vocab, d), 11, DEV, torch.bfloat16, scale=0.5)
    P = synth.randn((n, d), 12, DEV, torch.bfloat16, scale=0.5) if pos else None
    g = (1 + 0.1 * synth.randn((d,), 13, DEV, torch.float32)) if affine else None
    b = (0.1 * synth.randn((d,), 14, DEV, torch.float32)) if affine else None
    tok = torch.randint(0, vocab, (S, n), generator=torch.Generator(device="cpu").manual_seed(15)).to(DEV)
    tok[0, 1] = vocab + 5                           # not a token of the table
    tok[S - 1, n - 1] = -3
    h0 = torch.full((S, n, d), 7.0, dtype=torch.bfloat16, device=DEV)
    bad = torch.zeros(1, dtype=torch.int32, device=DEV)
    L.llmcache_embed(tok, E, P, h0, layer_norm=ln, ln_gain=g, ln_bias=b, eps=1e-5, bad_ids=bad)
    torch.cuda.synchronize()
    assert int(bad[0]) == 2
    exact = T.embed_f64(tok.cpu().numpy(), synth.bf16_bits(E), synth.bf16_bits(P) if pos else None, ln,
                        None if g is None else g.cpu().numpy(), None if b is None else b.cpu().numpy(), 1e-5)
    want = O.bf16_round(exact.astype(np.float32))
    got = synth.bf16_bits(h0)
    assert not got[0, 1].any() and not got[S - 1, n - 1].any()
    gf, wf = O.bf16_to_f32(got).astype(np.float64), O.bf16_to_f32(want).astype(np.float64)
    step = np.maximum(np.abs(wf), 2.0 ** -126) * 2.0 ** -7         # one bf16 step at that magnitude, at most
    assert np.all(np.abs(gf - wf) <= step)
    assert np.mean(got != want) <= 0.01
    if not ln:
        assert np.array_equal(got, want)            # a sum of two bf16 numbers, rounded once: the same bits


def test_embed_argument_errors_and_empty_batch():
    E = synth.randn((10, 64), 1, DEV, torch.bfloat16)
    tok = torch.zeros((2, 4), dtype=torch.int64, device=DEV)
    h0 = torch.zeros((2, 4, 64), dtype=torch.bfloat16, device=DEV)
    L.llmcache_embed(tok[:0], E, None, h0[:0])      # nothing to do
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_embed(tok, synth.randn((10, 60), 1, DEV, torch.bfloat16), None,
                         torch.zeros((2, 4, 60), dtype=torch.bfloat16, device=DEV))
    assert e.value.status == L.ERR_SHAPE
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_embed(tok, E, None, h0.view(-1)[1:])          # two bytes past a 16-byte boundary
    assert e.value.status == L.ERR_ARG
