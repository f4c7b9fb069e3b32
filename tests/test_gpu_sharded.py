"""A bank split into parts (the lookup half of sharing one cache between GPUs), with all parts on one GPU.

The parts are scanned one after the other into the same best words -- the same 64-bit maximum that an
all-reduce takes between GPUs -- so one GPU is enough to check the kernels: the split lookup must give the
oracle's decisions, slots and scores over the whole bank, bit-identical flags and index lists in every part,
the stored rows of the hits, and a metadata refresh that lands in the part that owns the matched slot; misses
shared out over the parts must be found again, by any part's scan, at the slots of the whole bank.
"""
import numpy as np
import pytest
import torch

from oracle import llmcache_oracle as O
from paper_2512_16843_b200 import binding as L
from paper_2512_16843_b200 import sharded as S
from paper_2512_16843_b200 import synth
from tests import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"


def whole_bank_oracle(sb: S.ShardedBank, n, k) -> O.Bank:
    """An oracle bank of n_total slots holding the parts' contents side by side."""
    ob = O.Bank(capacity=sb.n_total, seq_len=n, d_model=k, fp_dim=k, tau=0.9, policy=O.POLICY_LRU_STALENESS)
    cat = lambda what, conv: np.concatenate([conv(p.export(what)) for p in sb.parts])
    ob.fp = cat(L.WHAT_FP, U.bits)
    ob.rb = cat(L.WHAT_RB, lambda t: t.numpy().copy())
    ob.valid = cat(L.WHAT_VALID, lambda t: t.numpy().copy())
    ob.last_use = cat(L.WHAT_LAST_USE, U.u32)
    ob.insert_tick = cat(L.WHAT_INSERT_TICK, U.u32)
    ob.hits = cat(L.WHAT_HITS, U.u32)
    ob.m = cat(L.WHAT_RATE, U.u32)
    ob.e_upd = cat(L.WHAT_RATE_EPOCH, U.u32)
    ob.act = cat(L.WHAT_ACT, U.bits)
    ob.tick = int(sb.parts[0].export(L.WHAT_TICK)[0])
    return ob


@pytest.mark.parametrize("n_total,world,B", [(3001, 3, 300), (640, 2, 70), (5000, 4, 2500)])
def test_split_bank_lookup_and_shared_inserts_match_the_oracle(n_total, world, B):
    n, k = 2, 128
    sb = S.ShardedBank(n_total, world, list(range(world)), seq_len=n, d_model=k, fp_dim=k, max_batch=B, tau=0.9)
    keys, q, src = synth.scan_stress(n_total, B, k, n_clusters=64, seed=91 + n_total, device=DEV)
    acts = synth.activations(n_total, n, k, 17, DEV)
    valid = (synth.randn((n_total,), 5, "cpu") > -1.2).to(torch.uint8)
    rb = torch.from_numpy(O.inv_norm_of_stored(U.bits(keys)))
    for p, first in zip(sb.parts, sb.base):
        sl = slice(first, first + p.N)
        p.import_(L.WHAT_FP, keys[sl]); p.import_(L.WHAT_RB, rb[sl]); p.import_(L.WHAT_VALID, valid[sl])
        p.import_(L.WHAT_ACT, acts[sl])
    bufs = L.ProbeBuffers(B, k, DEV)
    sentinel = 0x7FC1
    for step in range(3):
        ob = whole_bank_oracle(sb, n, k)
        qs = q if step < 2 else synth.randn((B, k), 300, DEV, torch.bfloat16)      # third step: all fresh, all miss
        bufs.fp[:B].copy_(qs)
        h_out = torch.zeros((B, n * k), dtype=torch.bfloat16, device=DEV)
        h_out.view(torch.int16).fill_(sentinel)
        sb.probe_fp(bufs, B, h_out=h_out)
        torch.cuda.synchronize()
        assert all(p.status() == L.OK for p in sb.parts)
        qb = U.bits(qs)
        pr = O.probe_fp(ob, qb, O.inv_norm_of_stored(qb), 0.9, None, keep_scores=True)
        near_thr, near_tie = U.compare_probe(pr, bufs, B, 0.9)
        H, M = int(bufs.counts[0]), int(bufs.counts[1])
        if step == 0:
            assert H >= int((src >= 0).sum()) // 2 and M > 0
        elif step == 1:
            assert H == B                                 # the first step's misses were stored: everything is found
        else:
            assert H == 0
        # gathered rows: every hit's stored row, whichever part owns it; miss rows untouched
        out = U.bits(h_out)
        slot = bufs.slot[:B].cpu().numpy()
        for b in range(B):
            if slot[b] >= 0:
                assert np.array_equal(out[b], ob.act[slot[b]]), f"row {b}"
            else:
                assert np.all(out[b] == sentinel)
        # metadata refresh: the oracle touched its whole bank; every part must hold its slice of the result
        # (when a decision or a slot differed within the tolerance the oracle touched other slots: skip then)
        if near_thr == 0 and near_tie == 0:
            now = whole_bank_oracle(sb, n, k)
            occ = ob.valid != 0
            for name in ("last_use", "hits", "m", "e_upd"):
                assert np.array_equal(getattr(now, name)[occ], getattr(ob, name)[occ]), name
        # the misses are stored, miss m by part m mod world; every one of them gets a slot of the whole bank
        mo = synth.activations(max(M, 1), n, k, 400 + step, DEV)[:M]
        res = sb.commit(mo, bufs, h_out=h_out)
        torch.cuda.synchronize()
        taken = torch.cat([v for _, v in res.values()]).cpu().numpy() if M else np.zeros(0, dtype=np.int64)
        assert len(taken) == M and len(set(taken[taken >= 0].tolist())) == int((taken >= 0).sum())
        for r, (pos, slots) in res.items():
            first, count = S.slice_bounds(n_total, world, r)
            s_ = slots.cpu().numpy()
            assert np.all((s_ == -1) | ((s_ >= first) & (s_ < first + count)))
        last_miss_idx = bufs.miss_idx[:M].cpu().numpy()
        if M:
            assert np.array_equal(U.bits(h_out)[last_miss_idx], U.bits(mo))
    # after the third commit: the fresh queries are found again, each at the slot its miss was given
    bufs.fp[:B].copy_(qs)
    h2 = torch.zeros((B, n * k), dtype=torch.bfloat16, device=DEV)
    sb.probe_fp(bufs, B, h_out=h2)
    torch.cuda.synchronize()
    hit = bufs.hit[:B].cpu().numpy().astype(bool)
    given = np.full(B, -1, dtype=np.int64)                                # slot of the whole bank each query's miss took
    miss_list = last_miss_idx
    for r, (pos, slots) in res.items():
        given[miss_list[pos.cpu().numpy()]] = slots.cpu().numpy()
    assert np.array_equal(hit, given >= 0)                               # found again iff it was stored
    assert np.allclose(bufs.score[:B].cpu().numpy()[hit], 1.0, atol=2e-3)
    assert np.array_equal(bufs.slot[:B].cpu().numpy()[hit], given[hit])
    assert np.array_equal(U.bits(h2)[hit], U.bits(mo)[np.searchsorted(miss_list, np.flatnonzero(hit))])
    sb.close()
