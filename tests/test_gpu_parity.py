"""GPU-vs-oracle parity through the C ABI (element by element, same seeded inputs)."""
import numpy as np
import pytest
import torch

from oracle import llmcache_oracle as O
from paper_2512_16843_b200 import binding as L
from paper_2512_16843_b200 import synth
from tests import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_pair(N, n, d, k, B, dtype="bf16", proj=None, center=None, **kw):
    gb = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B,
                hidden_dtype=L.BF16 if dtype == "bf16" else L.F32, proj=proj, center=center, **kw)
    ob = U.oracle_bank_like(gb, proj, center)
    return gb, ob


def rand_h(B, n, d, seed, dtype):
    return synth.randn((B, n, d), seed, DEV, torch.bfloat16 if dtype == "bf16" else torch.float32)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(1, 1, 64, 1), (3, 5, 64, 7), (100, 37, 128, 33), (257, 130, 192, 65)])
def test_small_and_ragged_shapes_lockstep(shape, dtype):
    N, n, d, B = shape
    gb, ob = make_pair(N, n, d, d, B, dtype)
    bufs = L.ProbeBuffers(B, d, DEV)
    base = rand_h(B, n, d, 11, dtype)
    for step in range(4):
        h = base.clone()
        if step >= 1:                                  # half repeats (hits), half new
            h[B // 2:] = rand_h(B - B // 2, n, d, 100 + step, dtype)
        mo = synth.activations(B, n, d, 500 + step, DEV)
        r = U.lockstep_step(gb, ob, bufs, h, dtype, mo)
        if step == 0:
            assert r["H"] == 0
        if step >= 1 and N >= B:
            assert r["H"] >= B // 2
    gb.close()


@pytest.mark.parametrize("k,use_center", [(768, False), (256, False), (256, True)])
def test_config1_single_layer_probe(k, use_center):
    """d_model 768, seq_len 128, fp32 hidden states, 1024 entries from 16 centres, 64 queries, tau 0.9."""
    N, n, d, B = 1024, 128, 768, 64
    proj = synth.projection(d, k, 77, DEV) if k != d else None
    center = synth.randn((d,), 78, DEV, scale=0.01) if use_center else None
    gb, ob = make_pair(N, n, d, k, B, "f32", proj, center, tau=0.9)
    wl = synth.ClusterWorkload(16, n, d, synth.BASE_SEED + 1000, DEV)
    bufs = L.ProbeBuffers(B, k, DEV)
    for first in range(0, N, B):                       # warm the bank through the library itself
        h = wl.entries(first, B)
        gb.probe(h, bufs)
        gb.commit(synth.activations(B, n, d, 9000 + first, DEV), bufs)
    torch.cuda.synchronize()
    assert gb.stats()["resident"] > 0
    h, src = wl.queries(B, N, synth.BASE_SEED + 1001)
    r = U.lockstep_step(gb, ob, bufs, h, "f32", synth.activations(B, n, d, 4242, DEV))
    # by construction the 32 near queries hit (cosine ~0.9987) and the 32 fresh ones miss
    hit = bufs.hit[:B].cpu().numpy().astype(bool)
    assert np.array_equal(hit, (src >= 0).cpu().numpy()), r
    assert r["near_thr"] == 0
    gb.close()


@pytest.mark.parametrize("policy", [L.LRU, L.LRU_STALENESS])
def test_churn_lockstep_many_batches(policy):
    """Drifting centres, junk that never repeats, continuous eviction (small stand-in of the churn config)."""
    N, n, d, B = 64, 16, 128, 48
    gb, ob = make_pair(N, n, d, d, B, "bf16", policy=policy, half_life_ticks=2, min_age_ticks=2)
    bufs = L.ProbeBuffers(B, d, DEV)
    centres = synth.randn((16, n, d), 5, DEV)
    tot = dict(near_thr=0, near_tie=0, H=0, inserted=0)
    for step in range(24):
        centres = centres + synth.randn(centres.shape, 600 + step, DEV, scale=0.02)
        pick = torch.randint(0, 16, (36,), generator=torch.Generator().manual_seed(step)).to(DEV)
        near = centres[pick] + synth.randn((36, n, d), 700 + step, DEV, scale=0.05)
        junk = synth.randn((12, n, d), 800 + step, DEV)
        h = torch.cat([near, junk])[synth.shuffled(B, 900 + step, DEV)].to(torch.bfloat16).contiguous()
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 1000 + step, DEV))
        for key in tot:
            tot[key] += r[key]
    assert tot["H"] > 200 and tot["inserted"] > 200
    st = gb.stats()
    assert st["evictions"] > 0 and st["resident"] <= N
    gb.close()


def test_large_bank_eviction_path_lockstep():
    """More than 2048 slots: victim selection takes the radix-select path; must match the oracle's order."""
    N, n, d, B = 2500, 2, 64, 300
    gb, ob = make_pair(N, n, d, d, B, "bf16", half_life_ticks=2, min_age_ticks=1, stale_floor_q8=200)
    bufs = L.ProbeBuffers(B, d, DEV)
    hot = rand_h(100, n, d, 77, "bf16")
    inserted = 0
    for step in range(14):
        junk = rand_h(B - 100, n, d, 300 + step, "bf16")
        h = torch.cat([hot, junk])[synth.shuffled(B, 400 + step, DEV)].contiguous()
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 500 + step, DEV))
        inserted += r["inserted"]
    st = gb.stats()
    assert inserted > N and st["evictions"] > 0 and st["resident"] == N
    gb.close()


def test_probe_fp_path_and_act_rows_aliasing():
    N, k, B = 5000, 256, 300
    bank_fp, q, src = synth.scan_stress(N, B, k, n_clusters=128, seed=31, device=DEV)
    gb = L.Bank(capacity=N, seq_len=4, d_model=k, fp_dim=k, max_batch=B, act_rows=1000)
    ob = U.oracle_bank_like(gb)
    gb.import_(L.WHAT_FP, bank_fp)
    gb.import_(L.WHAT_RB, torch.from_numpy(O.inv_norm_of_stored(U.bits(bank_fp))))
    valid = torch.ones(N, dtype=torch.uint8)
    valid[::17] = 0
    gb.import_(L.WHAT_VALID, valid)
    gb.import_(L.WHAT_ACT, synth.activations(1000, 4, k, 3, DEV))
    bufs = L.ProbeBuffers(B, k, DEV)
    r = U.lockstep_step(gb, ob, bufs, q, "bf16", None, fp_only=True, do_commit=False)
    assert r["H"] > 30
    with pytest.raises(L.LLMCacheError) as e:
        gb.commit(synth.activations(B, 4, k, 4, DEV), bufs)
    assert e.value.status == L.ERR_UNSUPPORTED
    gb.close()


@pytest.mark.parametrize("N,k,B", [(20000, 1024, 1000), (3000, 64, 130), (70000, 128, 40), (513, 512, 257),
                                   (8192, 256, 512), (9000, 192, 300)])
def test_scan_many_tiles_and_runs(N, k, B):
    """Key counts and batch sizes that span many tensor-core tiles, several runs per block and ragged tails."""
    bank_fp, q, src = synth.scan_stress(N, B, k, n_clusters=64, seed=41 + k, device=DEV)
    gb = L.Bank(capacity=N, seq_len=2, d_model=k, fp_dim=k, max_batch=B, act_rows=512)
    ob = U.oracle_bank_like(gb)
    gb.import_(L.WHAT_FP, bank_fp)
    gb.import_(L.WHAT_RB, torch.from_numpy(O.inv_norm_of_stored(U.bits(bank_fp))))
    valid = (synth.randn((N,), 5, "cpu") > -1.0).to(torch.uint8)
    gb.import_(L.WHAT_VALID, valid)
    gb.import_(L.WHAT_ACT, synth.activations(512, 2, k, 3, DEV))
    bufs = L.ProbeBuffers(B, k, DEV)
    r = U.lockstep_step(gb, ob, bufs, q, "bf16", None, fp_only=True, do_commit=False)
    assert r["H"] > 0 and r["M"] > 0
    # duplicate keys: an exact tie must resolve to the lowest slot
    dup = bank_fp.clone()
    dup[N // 2:] = bank_fp[: N - N // 2]
    gb.import_(L.WHAT_FP, dup)
    gb.import_(L.WHAT_RB, torch.from_numpy(O.inv_norm_of_stored(U.bits(dup))))
    gb.import_(L.WHAT_VALID, torch.ones(N, dtype=torch.uint8))
    r = U.lockstep_step(gb, ob, bufs, dup[N // 2: N // 2 + B].contiguous(), "bf16", None, fp_only=True, do_commit=False)
    assert r["near_tie"] == 0 and r["H"] == B
    half = min(B, N // 2)
    assert bufs.slot[:half].cpu().tolist() == list(range(half))
    gb.close()


def test_empty_batch_degenerate_rows_and_miss_input_compaction():
    N, n, d, B = 16, 8, 64, 12
    gb, ob = make_pair(N, n, d, d, B, "f32")
    h_miss = torch.zeros((B, n, d), dtype=torch.float32, device=DEV)
    bufs = L.ProbeBuffers(B, d, DEV, h_miss=h_miss)
    gb.probe(torch.zeros((0, n, d), device=DEV), bufs, B=0)
    gb.commit(None, bufs)
    torch.cuda.synchronize()
    assert bufs.counts.tolist() == [0, 0] and int(gb.export(L.WHAT_TICK)[0]) == 1
    h = rand_h(B, n, d, 21, "f32")
    h[2] = 0.0
    h[5, 3, 7] = float("nan")
    h[7, 0, 0] = float("inf")
    mo = synth.activations(B, n, d, 22, DEV)
    r = U.lockstep_step(gb, ob, bufs, h, "f32", mo)
    assert r["H"] == 0 and r["inserted"] == B - 3
    assert torch.equal(h_miss.view(torch.int32), h.view(torch.int32))          # all miss: identity compaction
    r = U.lockstep_step(gb, ob, bufs, h, "f32", mo)
    assert r["H"] == B - 3
    mi = bufs.miss_idx[:3].long()
    assert mi.tolist() == [2, 5, 7]
    assert torch.equal(h_miss[:3].view(torch.int32), h[mi].view(torch.int32))
    st = gb.stats()
    assert st["degenerate"] == 6 and st["hits"] == B - 3 and st["sequences"] == 2 * B
    gb.close()


def test_threshold_modes_and_tau_sweep_monotone():
    N, n, d, B = 32, 4, 64, 32
    onehot = torch.zeros((B, n, d), device=DEV)
    for b in range(B):
        onehot[b, :, b] = 1.0
    for cmp, expect in ((L.GT, 0), (L.GE, B)):
        gb, ob = make_pair(N, n, d, d, B, "f32", cmp=cmp)
        bufs = L.ProbeBuffers(B, d, DEV)
        U.lockstep_step(gb, ob, bufs, onehot, "f32", synth.activations(B, n, d, 1, DEV))
        gb.probe(onehot, bufs, tau=1.0)                 # one-hot keys score exactly 1.0
        torch.cuda.synchronize()
        assert int(bufs.counts[0]) == expect
        gb.commit(synth.activations(B, n, d, 1, DEV), bufs)
        gb.close()
    gb, ob = make_pair(256, 8, 128, 128, 64, "bf16")
    bufs = L.ProbeBuffers(64, 128, DEV)
    base = rand_h(64, 8, 128, 5, "bf16")
    U.lockstep_step(gb, ob, bufs, base, "bf16", synth.activations(64, 8, 128, 2, DEV))
    noisy = (base.float() + 0.45 * synth.randn(base.shape, 6, DEV)).to(torch.bfloat16)
    prev = None
    for tau in (0.5, 0.8, 0.85, 0.9, 0.95):
        r = U.lockstep_step(gb, ob, bufs, noisy, "bf16", None, tau=tau, do_commit=False)
        hit = bufs.hit[:64].cpu().numpy()
        if prev is not None:
            assert np.all(hit <= prev)
        prev = hit
    assert prev.sum() < 64
    gb.close()


def test_evict_modes_match_oracle():
    import copy
    N, n, d, B = 40, 4, 64, 10
    gb, ob = make_pair(N, n, d, d, B, "f32", half_life_ticks=2, min_age_ticks=2, max_idle_ticks=6)
    bufs = L.ProbeBuffers(B, d, DEV)
    items = [rand_h(B, n, d, 40 + i, "f32") for i in range(4)]
    for i in range(4):
        U.lockstep_step(gb, ob, bufs, items[i], "f32", synth.activations(B, n, d, i, DEV))
    for _ in range(8):
        U.lockstep_step(gb, ob, bufs, items[1], "f32", synth.activations(B, n, d, 9, DEV))
    count = torch.zeros(1, dtype=torch.int32, device=DEV)
    U.pull_state(gb, ob)
    for mode in (L.EVICT_STALE, L.EVICT_IDLE):
        g2 = copy.deepcopy(ob)
        want = O.evict(g2, mode)
        saved = gb.export(L.WHAT_VALID)
        gb.evict(mode, count=count)
        torch.cuda.synchronize()
        assert int(count) == want and want > 0
        assert np.array_equal(gb.export(L.WHAT_VALID).numpy(), g2.valid)
        gb.import_(L.WHAT_VALID, saved)
    slots = torch.tensor([3, 3, 11, 39, -1, 400], dtype=torch.int32, device=DEV)
    gb.evict(L.EVICT_SLOTS, slots=slots, count=count)
    torch.cuda.synchronize()
    want = O.evict(ob, O.EVICT_SLOTS, [3, 3, 11, 39, -1, 400])
    assert int(count) == want and np.array_equal(gb.export(L.WHAT_VALID).numpy(), ob.valid)
    gb.evict(L.EVICT_ALL, count=count)
    torch.cuda.synchronize()
    assert int(count) == O.evict(ob, O.EVICT_ALL) and gb.stats()["resident"] == 0
    gb.close()


def test_call_order_and_argument_errors():
    gb, _ = make_pair(8, 4, 64, 64, 4, "f32")
    bufs = L.ProbeBuffers(4, 64, DEV)
    with pytest.raises(L.LLMCacheError) as e:
        gb.commit(synth.activations(4, 4, 64, 1, DEV), bufs)          # no probe yet
    assert e.value.status == L.ERR_STATE
    h = rand_h(4, 4, 64, 1, "f32")
    gb.probe(h, bufs)
    gb.commit(synth.activations(4, 4, 64, 1, DEV), bufs)
    with pytest.raises(L.LLMCacheError) as e:
        gb.commit(synth.activations(4, 4, 64, 1, DEV), bufs)          # committed twice
    assert e.value.status == L.ERR_STATE
    with pytest.raises(L.LLMCacheError) as e:
        gb.probe(rand_h(5, 4, 64, 1, "f32"), bufs)                     # B > max_batch
    assert e.value.status == L.ERR_SHAPE
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_probe(gb.handle, None, 4, None, None, bufs.io)       # null input
    assert e.value.status == L.ERR_ARG
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_probe(gb.handle, h.data_ptr() + 4, 4, None, None, bufs.io)   # misaligned
    assert e.value.status == L.ERR_ARG
    assert gb.status() == L.OK
    gb.close()


def test_arena_supplied_by_caller_and_repeatability():
    desc = L.make_desc(capacity=64, seq_len=8, d_model=64, fp_dim=64, max_batch=16, hidden_dtype=L.BF16)
    need = L.llmcache_bank_bytes(desc)
    arena = torch.empty(need + 256, dtype=torch.uint8, device=DEV)
    off = (-arena.data_ptr()) % 256
    outs = []
    for rep in range(2):
        gb = L.Bank(capacity=64, seq_len=8, d_model=64, fp_dim=64, max_batch=16, hidden_dtype=L.BF16,
                    arena=arena.data_ptr() + off, arena_bytes=need)
        bufs = L.ProbeBuffers(16, 64, DEV)
        h = rand_h(16, 8, 64, 3, "bf16")
        gb.probe(h, bufs)
        gb.commit(synth.activations(16, 8, 64, 4, DEV), bufs)
        gb.probe(h, bufs)
        torch.cuda.synchronize()
        outs.append((bufs.score.clone(), bufs.slot.clone(), bufs.fp.clone()))
        gb.close()
    assert all(torch.equal(a, b) for a, b in zip(outs[0], outs[1]))      # same bits on every run
    with pytest.raises(L.LLMCacheError) as e:
        L.Bank(capacity=64, seq_len=8, d_model=64, fp_dim=64, max_batch=16, arena=arena.data_ptr() + off, arena_bytes=1024)
    assert e.value.status == L.ERR_NOMEM


@pytest.mark.parametrize("N,n,d,k,B", [(300, 8, 128, 128, 70), (2048, 4, 768, 256, 256)])
def test_simhash_probe_matches_oracle_bit_for_bit(N, n, d, k, B):
    """SimHash lookup is integer work on the sign codes of the fingerprints: distances, slots, flags, gathered
    rows and metadata must match the oracle exactly (the oracle is given the GPU's query fingerprints, which
    are checked against its own within the usual tolerance); the reported angle estimate within 1e-6."""
    proj = synth.projection(d, k, 3, DEV) if k != d else None
    gb, ob = make_pair(N, n, d, k, B, "bf16", proj, None, tau=0.8)
    bufs = L.ProbeBuffers(B, k, DEV)
    base = rand_h(B, n, d, 61, "bf16")
    for step in range(3):
        h = base.clone()
        if step:                                         # two thirds noisy repeats, one third new
            h[: 2 * B // 3] = (base[: 2 * B // 3].float() + 0.15 * synth.randn((2 * B // 3, n, d), 70 + step, DEV)).to(torch.bfloat16)
            h[2 * B // 3:] = rand_h(B - 2 * B // 3, n, d, 80 + step, "bf16")
        U.pull_state(gb, ob)
        h_out = torch.zeros((B, n * d), dtype=torch.bfloat16, device=DEV)
        L.llmcache_probe_simhash(gb.handle, h, B, None, h_out, bufs.io)
        torch.cuda.synchronize()
        fq, rq = O.fingerprint(U.bits(h), "bf16", ob.proj, ob.center)
        U.compare_fingerprints(U.bits(bufs.fp[:B]), bufs.rq[:B].cpu().numpy(), fq, rq)
        exp_out = np.zeros((B, n * d), dtype=np.uint16)
        pr, ham = O.probe_simhash(ob, U.bits(bufs.fp[:B]), bufs.rq[:B].cpu().numpy(), 0.8, exp_out)
        assert np.array_equal(bufs.hit[:B].cpu().numpy(), pr.hit)
        assert np.array_equal(bufs.slot[:B].cpu().numpy(), pr.slot)
        assert np.allclose(bufs.score[:B].cpu().numpy(), pr.score, rtol=0, atol=1e-6)
        H = int(pr.hit.sum())
        assert bufs.counts.tolist() == [H, B - H]
        assert np.array_equal(U.bits(h_out), exp_out)
        U.assert_state_equal(gb, ob, with_act=False, where="after simhash probe")
        mo = synth.activations(B, n, d, 90 + step, DEV)
        gb.commit(mo, bufs, h_out=h_out)
        torch.cuda.synchronize()
        gp = U.gpu_probe_result(bufs, B, ob.tick)
        new = O.commit(ob, gp, U.bits(mo[:B - H]), exp_out)
        assert np.array_equal(bufs.new_slot[:B - H].cpu().numpy(), new)
        U.assert_state_equal(gb, ob, where="after commit")
        if step:
            assert 0 < H < B
    gb.close()


@pytest.mark.parametrize("dtype,d,k", [("bf16", 7680, 2048), ("f32", 3840, 2048), ("bf16", 2048, 2048)])
def test_maximum_widths(dtype, d, k):
    """Largest d_model per input type and largest fingerprint width, with and without a projection."""
    N, n, B = 33, 5, 9
    proj = synth.projection(d, k, 17, DEV) if k != d else None
    gb, ob = make_pair(N, n, d, k, B, dtype, proj, None)
    bufs = L.ProbeBuffers(B, k, DEV)
    base = rand_h(B, n, d, 19, dtype)
    for step in range(3):
        h = base.clone()
        if step:
            h[B // 2:] = rand_h(B - B // 2, n, d, 23 + step, dtype)
        r = U.lockstep_step(gb, ob, bufs, h, dtype, synth.activations(B, n, d, 29 + step, DEV))
    assert r["H"] >= B // 2
    for bad in (7688, 8192):
        with pytest.raises(L.LLMCacheError) as e:
            L.Bank(capacity=4, seq_len=2, d_model=bad, fp_dim=bad if bad <= 2048 else 2048, max_batch=2,
                   proj=synth.projection(bad, 2048, 1, DEV))
        assert e.value.status == L.ERR_SHAPE
    gb.close()


def test_large_batch_many_queries_per_slot_lockstep():
    """A batch that the decision kernel walks in several passes (more than 1,024 sequences), in which a few
    stored entries are matched by hundreds of queries each: the per-slot match counts, the decayed rates and
    the recency stamps must come out exactly as the oracle's, whichever thread applies them."""
    N, n, d, B = 1200, 2, 64, 2500               # the 1,000 misses of a step leave the 40 hot entries in the bank
    gb, ob = make_pair(N, n, d, d, B, "bf16", policy=L.LRU_STALENESS)
    bufs = L.ProbeBuffers(B, d, DEV)
    seeds = rand_h(40, n, d, 71, "bf16")
    g = torch.Generator().manual_seed(72)
    for step in range(3):
        h = rand_h(B, n, d, 80 + step, "bf16")
        if step:
            # 60% of the batch repeats one of 40 sequences that are in the bank after the first step
            rep = torch.randperm(B, generator=g)[: (B * 6) // 10].to(DEV)
            pick = torch.randint(0, 40, (rep.numel(),), generator=g).to(DEV)
            h[rep] = seeds[pick]
        else:
            h[:40] = seeds
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 90 + step, DEV))
        if step:
            assert r["H"] >= (B * 6) // 10
    assert int(ob.hits.max()) > 30
    gb.close()


@pytest.mark.parametrize("policy", [L.LRU, L.LRU_STALENESS])
def test_more_victims_than_the_shared_memory_sort_holds(policy):
    """Thousands of misses at once into a bank of thousands of slots: the chosen slots are sorted in pieces in
    shared memory and merged through global memory; which miss gets which slot must still be the oracle's."""
    N, n, d, B = 8000, 1, 64, 6000              # 6,000 inserts fill free slots first; later steps also evict thousands
    gb, ob = make_pair(N, n, d, d, B, "bf16", policy=policy)
    bufs = L.ProbeBuffers(B, d, DEV)
    keep = rand_h(700, n, d, 171, "bf16")
    for step in range(3):
        h = rand_h(B, n, d, 180 + step, "bf16")
        h[100:800] = keep                          # 700 sequences come back every step: their entries are hit and survive
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 190 + step, DEV))
        assert r["inserted"] == r["M"] > 2048
        if step:
            assert r["H"] >= 700
    gb.close()


@pytest.mark.parametrize("N,B,steps", [(5000, 20000, 3), (40000, 20000, 5), (262144, 65536, 7),
                                       (4097, 2049, 4), (8193, 8200, 3), (16390, 16385, 3)])
def test_large_bank_large_batch_commit_lockstep(N, B, steps):
    """Banks and batches for which the decision and the victim selection run as several grids: tens of
    thousands of misses per step take free slots first and then evict by (stale, decayed rate, last use, slot);
    the repeated keys are matched by several queries each.  Keys-only banks; the oracle scores a sample of
    the queries and replays the metadata refresh and the whole commit from the GPU's decisions."""
    k = 64
    gb = L.Bank(capacity=N, seq_len=1, d_model=k, fp_dim=k, max_batch=B, store_act=0, tau=0.9,
                policy=L.LRU_STALENESS, half_life_ticks=2, min_age_ticks=1, stale_floor_q8=200)
    ob = U.oracle_bank_like(gb, store_act=False)
    bufs = L.ProbeBuffers(B, k, DEV)
    g = torch.Generator().manual_seed(4242 + N)
    tot = dict(H=0, inserted=0)
    for step in range(steps):
        q = rand_h(B, 1, k, 9000 + 17 * step + N, "bf16").view(B, k)
        q = (q.float() / q.float().norm(dim=1, keepdim=True)).to(torch.bfloat16)
        resident = int(ob.valid.sum()) if step else 0
        if resident:
            # 40% of the batch repeats keys that are in the bank, drawn from a tenth of the occupied slots so
            # that many are matched several times
            occ = np.flatnonzero(ob.valid)
            pool_slots = occ[torch.randperm(len(occ), generator=g)[: max(1, len(occ) // 10)].numpy()]
            n_rep = (B * 4) // 10
            pick = pool_slots[torch.randint(0, len(pool_slots), (n_rep,), generator=g).numpy()]
            rows = torch.randperm(B, generator=g)[:n_rep].to(DEV)
            q[rows] = U.to_dev_bf16(ob.fp[pick], DEV)
        r = U.lockstep_step_sampled(gb, ob, bufs, q.contiguous(), 48, 77 + step)
        tot["H"] += r["H"]
        tot["inserted"] += r["inserted"]
        if resident:
            assert r["H"] >= (B * 4) // 10
    st = gb.stats()
    assert st["resident"] == min(N, tot["inserted"])
    if tot["inserted"] > N:
        assert st["evictions"] == tot["inserted"] - N
    if B > N:
        assert st["dropped"] > 0
    gb.close()
