"""Helpers for the GPU-vs-oracle parity tests: state transfer and comparisons.

Tolerances (floating point): fingerprints and scores must agree within 1e-3
relative (fp32 accumulation over bf16 / fp32 inputs against the oracle's
float64).  For a bf16 fingerprint "relative" is taken over the vector
(||gpu - oracle|| <= 1e-3 ||oracle||) and each element may differ by at most
one bf16 rounding step.  Decisions whose oracle score lies within 1e-3
(relative) of the threshold, and best-slot choices whose oracle scores differ
by less than 1e-3 (relative), are counted and reported, not failed.
Integer results (flags, indices, slots, metadata) and moved rows are bit-exact.
"""
import numpy as np
import torch

from oracle import llmcache_oracle as O
from paper_2512_16843_b200 import binding as L

REL = 1e-3


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def u32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().numpy().view(np.uint32)


def to_dev_bf16(bits_u16: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits_u16).view(np.int16).copy()).view(torch.bfloat16).to(device)


def oracle_bank_like(gb: L.Bank, proj=None, center=None, store_act=True) -> O.Bank:
    d = gb.desc
    return O.Bank(capacity=d.capacity, seq_len=d.seq_len, d_model=d.d_model, fp_dim=d.fp_dim,
                  act_rows=gb.act_rows, tau=float(d.tau), cmp_ge=(d.cmp == L.GE), policy=int(d.policy),
                  half_life_ticks=d.half_life_ticks or 8, stale_floor_q8=d.stale_floor_q8 or 64,
                  min_age_ticks=d.min_age_ticks or 4, max_idle_ticks=d.max_idle_ticks or 32,
                  proj=None if proj is None else bits(proj), center=None if center is None else center.cpu().numpy(),
                  store_act=store_act)


def pull_state(gb: L.Bank, ob: O.Bank, with_act=True):
    """Overwrite the oracle bank's state with the GPU bank's (lock-step)."""
    ob.fp = bits(gb.export(L.WHAT_FP))
    ob.rb = gb.export(L.WHAT_RB).numpy().copy()
    ob.valid = gb.export(L.WHAT_VALID).numpy().copy()
    ob.last_use = u32(gb.export(L.WHAT_LAST_USE)).copy()
    ob.insert_tick = u32(gb.export(L.WHAT_INSERT_TICK)).copy()
    ob.hits = u32(gb.export(L.WHAT_HITS)).copy()
    ob.m = u32(gb.export(L.WHAT_RATE)).copy()
    ob.e_upd = u32(gb.export(L.WHAT_RATE_EPOCH)).copy()
    ob.tick = int(gb.export(L.WHAT_TICK)[0])
    if with_act and ob.act is not None:
        ob.act = bits(gb.export(L.WHAT_ACT))


def assert_state_equal(gb: L.Bank, ob: O.Bank, with_act=True, where=""):
    assert int(gb.export(L.WHAT_TICK)[0]) == ob.tick, where
    valid = gb.export(L.WHAT_VALID).numpy()
    assert np.array_equal(valid, ob.valid), where + " valid"
    occ = ob.valid != 0
    for what, arr, name in ((L.WHAT_LAST_USE, ob.last_use, "last_use"), (L.WHAT_INSERT_TICK, ob.insert_tick, "insert_tick"),
                            (L.WHAT_HITS, ob.hits, "hits"), (L.WHAT_RATE, ob.m, "rate"),
                            (L.WHAT_RATE_EPOCH, ob.e_upd, "rate_epoch")):
        got = u32(gb.export(what))
        assert np.array_equal(got[occ], arr[occ]), f"{where} {name}"
    assert np.array_equal(bits(gb.export(L.WHAT_FP))[occ], ob.fp[occ]), where + " fp"
    assert np.array_equal(gb.export(L.WHAT_RB).numpy().view(np.uint32)[occ], ob.rb.view(np.uint32)[occ]), where + " rb"
    if with_act and ob.act is not None and gb.act_rows == gb.N:
        act = bits(gb.export(L.WHAT_ACT))
        assert np.array_equal(act[occ], ob.act[occ]), where + " act"


def compare_fingerprints(fp_gpu_bits, rq_gpu, fp_or_bits, rq_or):
    a = O.bf16_to_f32(fp_gpu_bits).astype(np.float64)
    b = O.bf16_to_f32(fp_or_bits).astype(np.float64)
    err = np.linalg.norm(a - b, axis=1)
    ref = np.linalg.norm(b, axis=1)
    assert np.all(err <= REL * np.maximum(ref, 1e-30) + 1e-12), f"fingerprint vector error {np.max(err / np.maximum(ref, 1e-30))}"
    assert np.all(np.abs(a - b) <= 2.0 ** -7 * np.abs(b) + 2e-6), "fingerprint element off by more than one rounding step"
    assert np.array_equal(rq_gpu == 0, rq_or == 0), "degenerate flags differ"
    assert np.allclose(rq_gpu, rq_or, rtol=REL, atol=0)
    return float((fp_gpu_bits != fp_or_bits).mean())


def compare_probe(pr: O.ProbeResult, bufs: L.ProbeBuffers, B, tau, cmp_ge=False):
    """Compare a GPU probe with the oracle's (run with keep_scores=True).  Returns counts of
    reported (not failed) near-threshold decisions and near-tie slot choices."""
    hit = bufs.hit[:B].cpu().numpy()
    slot = bufs.slot[:B].cpu().numpy()
    score = bufs.score[:B].cpu().numpy()
    counts = bufs.counts.cpu().numpy()
    H = int(counts[0]); M = int(counts[1])
    near_thr = 0
    near_tie = 0
    t32 = np.float32(tau)
    for b in range(B):
        so = float(pr.score[b]); sg = float(score[b])
        if np.isinf(so) or np.isinf(sg):
            assert so == sg, f"score[{b}] {sg} vs {so}"
        else:
            assert abs(sg - so) <= REL * max(abs(so), 1e-6) + 1e-6, f"score[{b}] {sg} vs {so}"
        if hit[b] != pr.hit[b]:
            assert abs(so - float(t32)) <= REL * abs(float(t32)) + 1e-6, f"decision[{b}] differs away from the threshold: {sg} vs {so}"
            near_thr += 1
            continue
        if hit[b]:
            if slot[b] != pr.slot[b]:
                assert pr.all_scores is not None
                alt = float(pr.all_scores[b, slot[b]])
                assert abs(alt - so) <= REL * abs(so), f"slot[{b}] {slot[b]} vs {pr.slot[b]}: {alt} vs {so}"
                near_tie += 1
        else:
            assert slot[b] == -1
    # compaction: consistent with the GPU's own flags, ascending, a partition
    hi = bufs.hit_idx[:H].cpu().numpy()
    mi = bufs.miss_idx[:M].cpu().numpy()
    assert H + M == B
    idx = np.arange(B, dtype=np.int32)
    assert np.array_equal(hi, idx[hit != 0]) and np.array_equal(mi, idx[hit == 0])
    if bufs.counts_host is not None:
        assert bufs.counts_host.tolist() == [H, M]
    return near_thr, near_tie


def gpu_probe_result(bufs: L.ProbeBuffers, B, tick) -> O.ProbeResult:
    """The GPU's probe outputs as an oracle ProbeResult (input of the oracle's commit step)."""
    counts = bufs.counts.cpu().numpy()
    H, M = int(counts[0]), int(counts[1])
    return O.ProbeResult(fp=bits(bufs.fp[:B]), rq=bufs.rq[:B].cpu().numpy(), score=bufs.score[:B].cpu().numpy(),
                         second=None, best_slot=None, hit=bufs.hit[:B].cpu().numpy(),
                         slot=bufs.slot[:B].cpu().numpy(), hit_idx=bufs.hit_idx[:H].cpu().numpy(),
                         miss_idx=bufs.miss_idx[:M].cpu().numpy(), tick=tick)


def assert_position_means(pooled_gpu: np.ndarray, h_bits: np.ndarray, n: int, d: int, where=""):
    """pooled_gpu [B, d] f32 against the exact means of the bf16 rows h_bits [B, n*d].  An fp32 sum of n
    terms in any order is off by at most (n - 1) * 2^-24 * sum|x|; the division adds one rounding."""
    x = O.bf16_to_f32(h_bits).astype(np.float64).reshape(h_bits.shape[0], n, d)
    want = x.mean(axis=1)
    bound = 2.0 * n * 2.0 ** -24 * np.abs(x).mean(axis=1) + 1e-30
    err = np.abs(pooled_gpu.astype(np.float64) - want)
    assert np.all(err <= bound), f"{where} position means off by {np.max(err / bound):.2f} x the bound"


def lockstep_step(gb: L.Bank, ob: O.Bank, bufs: L.ProbeBuffers, h_dev: torch.Tensor, dtype: str,
                  miss_out_dev: torch.Tensor, tau=None, with_act=True, fp_only=False, do_commit=True,
                  pooled_dev: torch.Tensor = None, before_commit=None):
    """One probe (+ commit) on both sides from the same state.  Returns dict of counters.
    pooled_dev: the GPU side probes from these position means instead of pooling h_dev itself (the
    oracle always starts from the hidden states: the result is defined to be the same)."""
    B = h_dev.shape[0]
    pull_state(gb, ob, with_act)
    n, d = gb.n, gb.d
    h_out = torch.zeros((max(B, 1), n * d), dtype=torch.bfloat16, device=h_dev.device)
    sentinel = 0x7FC1                      # a NaN pattern no generator produces
    h_out.view(torch.int16).fill_(sentinel)
    if fp_only:
        bufs.fp[:B].copy_(h_dev)
        gb.probe_fp(bufs, B, h_out=h_out, tau=tau)
    elif pooled_dev is not None:
        gb.probe_pooled(pooled_dev, bufs, B, h_out=h_out, tau=tau, h_in=h_dev)
    else:
        gb.probe(h_dev, bufs, h_out=h_out, tau=tau)
    torch.cuda.synchronize()
    assert gb.status() == L.OK
    tau_eff = float(gb.desc.tau) if tau is None else tau
    # oracle probe from the same state
    if fp_only:
        q = bits(h_dev)
        pr = O.probe_fp(ob, q, O.inv_norm_of_stored(q), tau_eff, None, keep_scores=True)
        flips = compare_fingerprints(bits(bufs.fp[:B]), bufs.rq[:B].cpu().numpy(), pr.fp, pr.rq) if B else 0.0
    else:
        host = h_dev.cpu()
        harr = bits(host) if dtype == "bf16" else host.numpy()
        pr = O.probe(ob, harr, dtype, tau_eff, None, keep_scores=True)
        flips = compare_fingerprints(bits(bufs.fp[:B]), bufs.rq[:B].cpu().numpy(), pr.fp, pr.rq) if B else 0.0
    near_thr, near_tie = compare_probe(pr, bufs, B, tau_eff, ob.cmp_ge)
    # gathered rows: verbatim copies of the stored rows of the GPU's slots; miss rows untouched
    gp = gpu_probe_result(bufs, B, ob.tick)
    if with_act and ob.act is not None and B:
        out = bits(h_out[:B])
        for b in range(B):
            if gp.hit[b]:
                assert np.array_equal(out[b], ob.act[int(gp.slot[b]) % ob.act_rows]), f"gathered row {b}"
            else:
                assert np.all(out[b] == sentinel), f"row {b} of a miss was written"
    # metadata after the probe: oracle touched with its own decisions; if some decisions were
    # reported as near-threshold/near-tie, re-touch from the pulled state with the GPU's slots
    if near_thr or near_tie:
        snap_tick = ob.tick
        pull_state(gb, ob, with_act=False)      # GPU state after its own touch
        ob.tick = snap_tick
    else:
        assert_state_equal(gb, ob, with_act=False, where="after probe")
    res = dict(near_thr=near_thr, near_tie=near_tie, H=len(gp.hit_idx), M=len(gp.miss_idx), fp_flips=flips)
    if not do_commit:
        return res
    M = len(gp.miss_idx)
    if before_commit is not None:
        # (stale-class slots, decayed entries) of the oracle's state as the commit will find it
        stale_set, res["decayed"] = before_commit(ob)
        was_valid = ob.valid.copy()
    h_out2 = h_out.clone()
    gb.commit(miss_out_dev, bufs, h_out=h_out2)
    torch.cuda.synchronize()
    assert gb.status() == L.OK
    mo = bits(miss_out_dev[:M]) if (with_act and M) else None
    ho = bits(h_out) if with_act else None
    new_or = O.commit(ob, gp, mo, ho)
    new_gpu = bufs.new_slot[:M].cpu().numpy()
    assert np.array_equal(new_gpu, new_or), f"new_slot {new_gpu} vs {new_or}"
    if before_commit is not None:
        res["stale_victims"] = sum(1 for v in new_or.tolist() if v >= 0 and was_valid[v] and v in stale_set)
    if with_act:
        assert np.array_equal(bits(h_out2), ho), "scattered outputs"
    assert_state_equal(gb, ob, with_act=with_act, where="after commit")
    res["inserted"] = int((new_or >= 0).sum())
    res["h_out"] = h_out2
    return res


def lockstep_step_sampled(gb: L.Bank, ob: O.Bank, bufs: L.ProbeBuffers, q_dev: torch.Tensor, n_sample: int, seed: int,
                          tau=None, do_commit=True):
    """One probe_fp (+ commit) of a keys-only bank that is too large for the oracle to score in full.
    The oracle scores a seeded sample of the queries against the whole bank (scores, decisions, slots);
    the compaction is checked in full against the GPU's own flags; the metadata refresh and the whole commit
    (which slots the misses take, every array of the bank afterwards) are the oracle's, computed from the
    GPU's decisions, and compared in full."""
    B = q_dev.shape[0]
    pull_state(gb, ob, with_act=False)
    bufs.fp[:B].copy_(q_dev)
    gb.probe_fp(bufs, B, tau=tau)
    torch.cuda.synchronize()
    assert gb.status() == L.OK
    tau_eff = float(gb.desc.tau) if tau is None else tau
    hit = bufs.hit[:B].cpu().numpy()
    slot = bufs.slot[:B].cpu().numpy()
    score = bufs.score[:B].cpu().numpy()
    H, M = [int(x) for x in bufs.counts.cpu()]
    assert H + M == B and H == int(hit.sum())
    idx = np.arange(B, dtype=np.int32)
    assert np.array_equal(bufs.hit_idx[:H].cpu().numpy(), idx[hit != 0])
    assert np.array_equal(bufs.miss_idx[:M].cpu().numpy(), idx[hit == 0])
    assert np.all(slot[hit == 0] == -1)
    # the oracle on a sample of the queries
    sample = np.sort(np.random.Generator(np.random.Philox(key=seed)).choice(B, min(n_sample, B), replace=False))
    qs = bits(q_dev[torch.from_numpy(sample).to(q_dev.device)])
    rqs = O.inv_norm_of_stored(qs)
    s = O.scores(qs, rqs, ob.fp, ob.rb, ob.valid)
    best, bslot, _ = O.best_match(s)
    ohit, oslot = O.decide(best, bslot, rqs, tau_eff, ob.cmp_ge)
    near = 0
    for i, b in enumerate(sample):
        so, sg = float(best[i]), float(score[b])
        if np.isinf(so) or np.isinf(sg):
            assert so == sg
        else:
            assert abs(sg - so) <= REL * max(abs(so), 1e-6) + 1e-6, f"score[{b}] {sg} vs {so}"
        if hit[b] != ohit[i]:
            assert abs(so - tau_eff) <= REL * abs(tau_eff) + 1e-6
            near += 1
        elif hit[b] and slot[b] != oslot[i]:
            assert abs(float(s[i, slot[b]]) - so) <= REL * abs(so)
            near += 1
    # metadata refresh from the GPU's decisions
    ob.tick += 1
    O.touch(ob, slot[hit != 0])
    assert_state_equal(gb, ob, with_act=False, where="after probe")
    res = dict(H=H, M=M, near=near)
    if not do_commit:
        return res
    gp = gpu_probe_result(bufs, B, ob.tick)
    gb.commit(None, bufs)
    torch.cuda.synchronize()
    assert gb.status() == L.OK
    new_or = O.commit(ob, gp, None, None)
    new_gpu = bufs.new_slot[:M].cpu().numpy()
    assert np.array_equal(new_gpu, new_or), "new_slot differs from the oracle's"
    assert_state_equal(gb, ob, with_act=False, where="after commit")
    res["inserted"] = int((new_or >= 0).sum())
    return res
