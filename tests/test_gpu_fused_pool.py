"""Fingerprint-on-write and the split fingerprint (pool / project) against the oracle.

The rows a layer writes (reused outputs copied out of the bank, computed outputs written back) are
summed on the way, so the next layer's probe starts from the position means instead of reading the
hidden states again.  Checked here: the moved rows and the bank state stay bit-exact, the means are
the exact means of the written rows within the fp32 summation bound, and a probe from those means
decides like the oracle's probe of the hidden states themselves.
"""
import numpy as np
import pytest
import torch

from oracle import llmcache_oracle as O
from paper_2512_16843_b200 import binding as L
from paper_2512_16843_b200 import synth
from tests import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"


def rand_h(B, n, d, seed):
    return synth.randn((B, n, d), seed, DEV, torch.bfloat16)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("B,n,d", [(1, 1, 64), (7, 5, 64), (50, 37, 768), (300, 130, 192)])
def test_pool_alone_matches_exact_means(B, n, d, dtype):
    gb = L.Bank(capacity=8, seq_len=n, d_model=d, fp_dim=d, max_batch=B,
                hidden_dtype=L.BF16 if dtype == "bf16" else L.F32)
    h = synth.randn((B, n, d), 5, DEV, torch.bfloat16 if dtype == "bf16" else torch.float32)
    # strided destination: the second half of a [B, 2d] array (the first half must stay untouched)
    pooled = torch.full((B, 2 * d), -7.0, dtype=torch.float32, device=DEV)
    gb.pool(h, pooled[:, d:])
    torch.cuda.synchronize()
    assert gb.status() == L.OK
    assert torch.all(pooled[:, :d] == -7.0)
    got = pooled[:, d:].cpu().numpy()
    if dtype == "bf16":
        U.assert_position_means(got, U.bits(h).reshape(B, n * d), n, d)
    else:
        x = h.cpu().numpy().astype(np.float64)
        bound = 2.0 * n * 2.0 ** -24 * np.abs(x).mean(axis=1) + 1e-30
        assert np.all(np.abs(got - x.mean(axis=1)) <= bound)
    assert np.allclose(got, O.pool(U.bits(h) if dtype == "bf16" else h.cpu().numpy(), dtype), rtol=0, atol=1e-5)
    gb.close()


@pytest.mark.parametrize("B,d,k,use_center", [(5, 64, 64, False), (130, 768, 256, True), (64, 1536, 256, False)])
def test_fingerprint_pooled_matches_oracle(B, d, k, use_center):
    proj = synth.projection(d, k, 3, DEV)
    center = synth.randn((d,), 4, DEV, scale=0.05) if use_center else None
    gb = L.Bank(capacity=8, seq_len=1, d_model=d, fp_dim=k, max_batch=B, proj=proj, center=center, store_act=0)
    p = synth.randn((B, d), 6, DEV, scale=0.3)
    p[B // 2].zero_()                                          # a degenerate row (only without centring)
    wide = torch.zeros((B, d + 16), dtype=torch.float32, device=DEV)
    wide[:, :d] = p
    fp = torch.empty((B, k), dtype=torch.bfloat16, device=DEV)
    rq = torch.empty((B,), dtype=torch.float32, device=DEV)
    gb.fingerprint_pooled(wide[:, :d], fp, rq)
    torch.cuda.synchronize()
    want_fp, want_rq = O.normalise(O.project(p.cpu().numpy().astype(np.float64), U.bits(proj),
                                             None if center is None else center.cpu().numpy()))
    U.compare_fingerprints(U.bits(fp), rq.cpu().numpy(), want_fp, want_rq)
    if not use_center:
        assert rq[B // 2].item() == 0.0
    gb.close()


def test_attention_augmented_fingerprint_matches_oracle():
    """Sec. IV-B bullet 2: position means of the embeddings and of the first self-attention output,
    side by side, projected by one [2d, k] matrix."""
    B, n, d, k = 40, 33, 256, 128
    proj = synth.projection(2 * d, k, 9, DEV)
    center = synth.randn((2 * d,), 10, DEV, scale=0.02)
    pool_bank = L.Bank(capacity=8, seq_len=n, d_model=d, fp_dim=d, max_batch=B, store_act=0)
    fp_bank = L.Bank(capacity=8, seq_len=n, d_model=2 * d, fp_dim=k, max_batch=B, proj=proj, center=center, store_act=0)
    h = rand_h(B, n, d, 21)
    attn = synth.randn((B, n, d), 22, DEV, torch.bfloat16, scale=0.5)
    pooled = torch.empty((B, 2 * d), dtype=torch.float32, device=DEV)
    pool_bank.pool(h, pooled[:, :d])
    pool_bank.pool(attn, pooled[:, d:])
    fp = torch.empty((B, k), dtype=torch.bfloat16, device=DEV)
    rq = torch.empty((B,), dtype=torch.float32, device=DEV)
    fp_bank.fingerprint_pooled(pooled, fp, rq)
    torch.cuda.synchronize()
    want_fp, want_rq = O.fingerprint_augmented(U.bits(h), "bf16", U.bits(attn), "bf16", U.bits(proj), center.cpu().numpy())
    U.compare_fingerprints(U.bits(fp), rq.cpu().numpy(), want_fp, want_rq)
    pool_bank.close()
    fp_bank.close()


@pytest.mark.parametrize("N,n,d,k,B", [(16, 1, 64, 64, 3), (64, 5, 64, 64, 20), (256, 37, 768, 256, 100),
                                       (300, 130, 192, 64, 257)])
def test_fused_pool_two_layer_chain_lockstep(N, n, d, k, B):
    """Two banks in a chain: bank 1 writes h_1 with the sums taken on the way, bank 2 probes from them.
    A sequence that repeats is served the stored row by bank 1, so bank 2 sees a repeated input too."""
    proj = synth.projection(d, k, 31, DEV) if k != d else None
    kw = dict(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, proj=proj, fused_pool=1)
    g1, g2 = L.Bank(**kw), L.Bank(**kw)
    o1, o2 = U.oracle_bank_like(g1, proj), U.oracle_bank_like(g2, proj)
    b1, b2 = L.ProbeBuffers(B, k, DEV), L.ProbeBuffers(B, k, DEV)
    pooled = torch.zeros((B, d + 8), dtype=torch.float32, device=DEV)[:, :d]      # rows 8 floats apart from dense
    base = rand_h(B, n, d, 41)
    g1.pool_out(pooled)
    seen = dict(H0=False, M0=False, hits2=0)
    for step in range(5):
        h0 = base.clone()
        if step in (1, 2):                               # half repeats, half new
            h0[B // 2:] = rand_h(B - B // 2, n, d, 200 + step)
        if step == 4:                                    # nothing repeats; step 3: everything does
            h0 = rand_h(B, n, d, 300)
        pooled.fill_(float("nan"))
        r1 = U.lockstep_step(g1, o1, b1, h0, "bf16", synth.activations(B, n, d, 600 + step, DEV))
        h1 = r1["h_out"]
        seen["H0"] |= r1["H"] == 0
        seen["M0"] |= r1["M"] == 0
        U.assert_position_means(pooled.cpu().numpy(), U.bits(h1[:B]), n, d, where=f"step {step}")
        r2 = U.lockstep_step(g2, o2, b2, h1[:B].view(B, n, d), "bf16", synth.activations(B, n, d, 700 + step, DEV),
                             pooled_dev=pooled)
        seen["hits2"] += r2["H"]
        if step == 0:
            assert r1["H"] == 0 and r2["H"] == 0
        if step == 1 and N >= 2 * B:
            assert r1["H"] >= B // 2 and r2["H"] >= B // 2
    assert seen["H0"] and seen["hits2"] > 0
    if N >= 2 * B:
        assert seen["M0"]
    assert g1.status() == L.OK and g2.status() == L.OK
    g1.close()
    g2.close()


def test_fused_pool_argument_and_order_errors():
    n, d, B = 4, 64, 8
    plain = L.Bank(capacity=16, seq_len=n, d_model=d, fp_dim=d, max_batch=B)
    pooled = torch.zeros((B, d), dtype=torch.float32, device=DEV)
    with pytest.raises(L.LLMCacheError) as e:
        plain.pool_out(pooled)                           # bank was not created for it
    assert e.value.status == L.ERR_UNSUPPORTED
    plain.close()
    with pytest.raises(L.LLMCacheError):
        L.Bank(capacity=16, seq_len=n, d_model=d, fp_dim=d, max_batch=B, fused_pool=1, store_act=0)
    gb = L.Bank(capacity=16, seq_len=n, d_model=d, fp_dim=d, max_batch=B, fused_pool=1)
    bufs = L.ProbeBuffers(B, d, DEV)
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_bank_pool_out(gb.handle, pooled, d - 1)
    assert e.value.status == L.ERR_SHAPE
    gb.pool_out(pooled)
    h = rand_h(B, n, d, 1)
    with pytest.raises(L.LLMCacheError) as e:
        gb.probe(h, bufs)                                # h_out is required while the sums are taken
    assert e.value.status == L.ERR_ARG
    h_out = torch.zeros((B, n * d), dtype=torch.bfloat16, device=DEV)
    gb.probe(h, bufs, h_out=h_out)
    with pytest.raises(L.LLMCacheError) as e:
        gb.pool_out(None)                                # not between a probe and its commit
    assert e.value.status == L.ERR_STATE
    gb.commit(synth.activations(B, n, d, 2, DEV), bufs, h_out=h_out)
    gb.pool_out(None)
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_probe_pooled(gb.handle, pooled, d - 8, None, B, None, h_out, bufs.io)
    assert e.value.status == L.ERR_SHAPE
    torch.cuda.synchronize()
    assert gb.status() == L.OK
    gb.close()
