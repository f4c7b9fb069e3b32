"""Parity at the full sizes of the five benchmark configurations, through the C ABI, in the same
launch configuration the benchmark times.  Where the oracle cannot afford the whole output (the
bank-scan stress) it is computed for a seeded sample of queries, and size-independent properties are
checked on the rest."""
import numpy as np
import pytest
import torch

from oracle import llmcache_oracle as O
from paper_2512_16843_b200 import binding as L
from paper_2512_16843_b200 import synth
from tests import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"
SEED = synth.BASE_SEED


def warm_through_library(gb, bufs, batches, n, d):
    for i, hb in enumerate(batches):
        gb.probe(hb, bufs)
        gb.commit(synth.activations(hb.shape[0], n, d, 7000 + i, DEV), bufs)
    torch.cuda.synchronize()


@pytest.mark.parametrize("k,centred", [(256, False), (256, True), (768, False)])
def test_config2_bert_base_shaped_layer(k, centred):
    """d_model 768, seq_len 384, batch 256 (60% token-level edits of 64 seeds), bank of 2048, tau 0.80/0.90/0.95."""
    N, n, d, B = 2048, 384, 768, 256
    wl = synth.TokenWorkload(30522, n, d, SEED + 2000, DEV)
    seeds_tok = wl.tokens(64, SEED + 2005)
    proj = synth.projection(d, k, SEED + 2006, DEV) if k != d else None
    center = None
    if centred:                                   # mean pooled vector of a seeded calibration batch (an input)
        calib = wl.hidden(wl.tokens(64, SEED + 2007))
        center = calib.float().mean(dim=(0, 1)).contiguous()
    gb = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, hidden_dtype=L.BF16, proj=proj,
                center=center, tau=0.9)
    ob = U.oracle_bank_like(gb, proj, center)
    bufs = L.ProbeBuffers(B, k, DEV)
    warm = [wl.hidden(torch.cat([seeds_tok, wl.tokens(B - 64, SEED + 2008)]))]
    warm += [wl.hidden(wl.tokens(B, SEED + 2020 + i)) for i in range(1, N // B)]
    warm_through_library(gb, bufs, warm, n, d)
    assert gb.stats()["resident"] == N
    n_edit = int(round(B * 0.6))
    ed, _ = wl.edited(seeds_tok, n_edit, 0.10, SEED + 2101)
    tok = torch.cat([ed, wl.tokens(B - n_edit, SEED + 2102)])[synth.shuffled(B, SEED + 2103, DEV)]
    h = wl.hidden(tok)
    report = {}
    for tau in (0.80, 0.90, 0.95):
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", None, tau=tau, do_commit=False)
        report[tau] = (r["H"], r["near_thr"], r["near_tie"])
    r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 99, DEV), tau=0.90)
    print("config2 k=%d centred=%s: (hits, near-threshold, near-tie) per tau %s; commit inserted %d"
          % (k, centred, report, r["inserted"]))
    assert report[0.80][0] >= report[0.90][0] >= report[0.95][0]
    if not centred:
        assert report[0.90][0] == n_edit            # edits score ~0.95, fresh ~0.5: tau 0.9 separates them
    gb.close()


def test_config3_gpt2_small_shaped_layer():
    """d_model 768, seq_len 1024, batch 32 sharing 512-token prefixes with 8 seed documents, bank of 1024."""
    N, n, d, B, k = 1024, 1024, 768, 32, 256
    wl = synth.TokenWorkload(50257, n, d, SEED + 3000, DEV)
    seeds_tok = wl.tokens(8, SEED + 3005)
    proj = synth.projection(d, k, SEED + 3006, DEV)
    gb = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, hidden_dtype=L.BF16, proj=proj, tau=0.9)
    ob = U.oracle_bank_like(gb, proj, None)
    bufs = L.ProbeBuffers(B, k, DEV)
    warm_tok = [wl.with_shared_prefix(seeds_tok, B, 512, SEED + 3100 + i)[0] for i in range(N // B)]
    warm_through_library(gb, bufs, [wl.hidden(t) for t in warm_tok], n, d)
    # measured batch: 16 exact repeats of warmed sequences (hit, score 1) + 16 new suffixes (miss)
    rep = torch.cat([warm_tok[3][:8], warm_tok[17][8:16]])
    new, _ = wl.with_shared_prefix(seeds_tok, 16, 512, SEED + 3999)
    tok = torch.cat([rep, new])[synth.shuffled(B, SEED + 3998, DEV)]
    r = U.lockstep_step(gb, ob, bufs, wl.hidden(tok), "bf16", synth.activations(B, n, d, 5, DEV))
    print("config3: hits %d, near-threshold %d, near-tie %d" % (r["H"], r["near_thr"], r["near_tie"]))
    assert r["H"] >= 16
    gb.close()


@pytest.mark.parametrize("N", [65536, 262144, 1048576])
def test_config4_bank_scan_stress_sampled(N):
    """fp_dim 1024, 65,536 queries against N keys from 4,096 clusters, 30% near-duplicates, top-1 + tau 0.9.
    The oracle scores a seeded sample of the queries against the whole bank."""
    B, k = 65536, 1024
    n_sample = 512 if N <= 65536 else 256 if N <= 262144 else 128
    keys, q, src = synth.scan_stress(N, B, k, n_clusters=4096, spread=0.1, near_fraction=0.3, q_sigma=0.05,
                                     seed=SEED + 4000, device=DEV)
    gb = L.Bank(capacity=N, seq_len=1, d_model=k, fp_dim=k, max_batch=B, store_act=0, tau=0.9)
    bufs = L.ProbeBuffers(B, k, DEV)
    for f in range(0, N, B):                       # fill through the library, as the benchmark does
        bufs.fp[:B].copy_(keys[f:f + B])
        gb.probe_fp(bufs, B, tau=2.0)
        gb.commit(None, bufs)
    torch.cuda.synchronize()
    assert gb.stats()["resident"] == N
    bufs.fp.copy_(q)
    gb.probe_fp(bufs, B)
    torch.cuda.synchronize()
    assert gb.status() == L.OK
    hit = bufs.hit.cpu().numpy()
    slot = bufs.slot.cpu().numpy()
    score = bufs.score.cpu().numpy()
    H, M = [int(x) for x in bufs.counts.cpu()]
    # properties that hold at any size
    assert H + M == B and H == int(hit.sum())
    idx = np.arange(B, dtype=np.int32)
    assert np.array_equal(bufs.hit_idx[:H].cpu().numpy(), idx[hit != 0])
    assert np.array_equal(bufs.miss_idx[:M].cpu().numpy(), idx[hit == 0])
    assert np.all(slot[hit == 0] == -1) and np.all((slot[hit != 0] >= 0) & (slot[hit != 0] < N))
    assert np.all(score <= 1.0 + 1e-5)
    # by construction: near-duplicates hit (cosine ~0.9988 against their source), fresh queries miss
    assert np.array_equal(hit != 0, (src >= 0).cpu().numpy())
    # the oracle on a seeded sample of the queries, against the full bank
    sample = np.sort(np.random.Generator(np.random.Philox(key=SEED + 4001)).choice(B, n_sample, replace=False))
    ob = O.Bank(capacity=N, seq_len=1, d_model=k, fp_dim=k, tau=0.9, store_act=False)
    U.pull_state(gb, ob, with_act=False)
    ob.tick -= 1                                   # state as of before the measured probe (a probe only ticks)
    qs = U.bits(q[torch.from_numpy(sample).to(DEV)])
    pr = O.probe_fp(ob, qs, O.inv_norm_of_stored(qs), 0.9, None, keep_scores=True)
    near_tie = 0
    for i, b in enumerate(sample):
        so, sg = float(pr.score[i]), float(score[b])
        assert abs(sg - so) <= U.REL * max(abs(so), 1e-6) + 1e-6
        assert hit[b] == pr.hit[i] or abs(so - 0.9) <= U.REL * 0.9
        if hit[b] and slot[b] != pr.slot[i]:
            assert abs(float(pr.all_scores[i, slot[b]]) - so) <= U.REL * abs(so)
            near_tie += 1
    print("config4 N=%d: %d hits of %d queries, %d sampled, %d near-ties" % (N, H, B, n_sample, near_tie))
    gb.close()


def test_config4_gather_of_one_mebibyte_rows():
    """Gather of hit rows of 512 x 1024 bf16 activations through an aliased activation pool (slot mod act_rows)."""
    N, B, k, n, act_rows = 65536, 2048, 1024, 512, 1024
    keys, q, src = synth.scan_stress(N, B, k, n_clusters=4096, seed=SEED + 4100, device=DEV)
    gb = L.Bank(capacity=N, seq_len=n, d_model=k, fp_dim=k, max_batch=B, act_rows=act_rows, tau=0.9)
    gb.import_(L.WHAT_FP, keys)
    gb.import_(L.WHAT_RB, torch.from_numpy(O.inv_norm_of_stored(U.bits(keys))))
    gb.import_(L.WHAT_VALID, torch.ones(N, dtype=torch.uint8))
    act = synth.activations(act_rows, n, k, 9, DEV)
    gb.import_(L.WHAT_ACT, act)
    bufs = L.ProbeBuffers(B, k, DEV)
    bufs.fp.copy_(q)
    h_out = torch.zeros((B, n * k), dtype=torch.bfloat16, device=DEV)
    gb.probe_fp(bufs, B, h_out=h_out)
    torch.cuda.synchronize()
    hit = bufs.hit.bool()
    slot = bufs.slot.long()
    assert int(hit.sum()) == int((src >= 0).sum())
    want = act[slot[hit] % act_rows]
    assert torch.equal(h_out[hit].view(torch.int16), want.view(torch.int16))
    assert not h_out[~hit].any()
    gb.close()


@pytest.mark.parametrize("layer", [1, 12, 24])
def test_config5_bert_large_shaped_churn_lockstep(layer):
    """d_model 1024, seq_len 512, batch 512, bank of 1024 with insert on miss and LRU + staleness eviction under
    drifting cluster centres (shift 0.02 per batch), junk that never repeats and topic turnover; lock-step.
    Three separately seeded banks (standing for layers 1, 12 and 24 of the encoder), each for 24 batches = three
    half-lives of the decayed match rate with the default policy constants; every batch is compared in full
    (decisions, gathered rows, which slot each miss takes, every array of the bank).  With the default constants
    the ~110 evictions per batch recycle every low-rate entry within about seven batches, before its rate has
    halved three times, so rates are seen decayed but no entry lives long enough to turn stale; the third bank
    therefore halves the rate every batch, which makes junk stale after four batches, and must take victims
    from the stale class."""
    N, n, d, B, k = 1024, 512, 1024, 512, 256
    n_centres = 256
    S = SEED + 97 * layer
    proj = synth.projection(d, k, S + 5006, DEV)
    gb = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, hidden_dtype=L.BF16, proj=proj, tau=0.9,
                policy=L.LRU_STALENESS, half_life_ticks=1 if layer == 24 else 0)
    ob = U.oracle_bank_like(gb, proj, None)
    bufs = L.ProbeBuffers(B, k, DEV)
    centres = synth.randn((n_centres, n, d), S + 5000, DEV, torch.bfloat16)
    g = torch.Generator().manual_seed(S + 5001)
    tot = dict(H=0, inserted=0, near_thr=0, near_tie=0)
    steps = 24
    stale_victims = 0
    decayed_seen = 0
    for step in range(steps):
        centres = (centres.float() + synth.randn(centres.shape, S + 5100 + step, DEV, scale=0.02)).to(torch.bfloat16)
        for c in torch.randint(0, n_centres, (2,), generator=g).tolist():      # topic turnover
            centres[c] = synth.randn((n, d), S + 5200 + 10 * step + c, DEV, torch.bfloat16)
        n_near = int(B * 0.75)
        pick = torch.randint(0, n_centres, (n_near,), generator=g).to(DEV)
        h = torch.empty((B, n, d), dtype=torch.bfloat16, device=DEV)
        for i0 in range(0, n_near, 64):
            sl = slice(i0, min(n_near, i0 + 64))
            h[sl] = (centres[pick[sl]].float() + synth.randn((sl.stop - sl.start, n, d), S + 5300 + 100 * step + i0,
                                                             DEV, scale=0.05)).to(torch.bfloat16)
        h[n_near:] = synth.randn((B - n_near, n, d), S + 5400 + step, DEV, torch.bfloat16)
        h = h[synth.shuffled(B, S + 5500 + step, DEV)].contiguous()
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, S + 5600 + step, DEV),
                            before_commit=lambda bank: stale_and_decayed(bank))
        stale_victims += r["stale_victims"]
        decayed_seen = max(decayed_seen, r["decayed"])
        for key in tot:
            tot[key] += r[key]
        del h
    st = gb.stats()
    print("config5 bank %d: %d steps, hits %d, inserted %d, evictions %d, stale-class victims %d, decayed entries (max) %d, "
          "near-threshold %d, near-tie %d" % (layer, steps, tot["H"], tot["inserted"], st["evictions"], stale_victims,
                                              decayed_seen, tot["near_thr"], tot["near_tie"]))
    assert st["evictions"] > 0 and tot["H"] > 0 and st["resident"] == N
    if layer == 24:
        assert stale_victims > 0, "no victim was ever taken from the stale class"
    assert decayed_seen > 0, "no stored entry's match rate was ever seen decayed"
    gb.close()


def stale_and_decayed(ob):
    """From the oracle bank's state between a probe and its commit: the slots in the stale class, and how many
    occupied entries carry a match rate that has decayed since it was last written."""
    occ = np.flatnonzero(ob.valid)
    stale = {int(j) for j in occ if O.is_stale(ob, int(j))}
    decayed = sum(1 for j in occ if O.effective_rate(ob, int(j)) < int(ob.m[j]))
    return stale, decayed
