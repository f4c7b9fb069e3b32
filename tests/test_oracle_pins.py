"""Pins for the CPU oracle: each test checks it against something that is not
the oracle itself -- exact rational arithmetic, a library routine, a textbook
simulation, a closed form, a hand-worked value, or brute force on tiny inputs.
"""
import collections
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy.spatial.distance import cdist

from oracle import llmcache_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.Generator(np.random.Philox(key=seed))


def torch_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """bfloat16 conversion by a library (torch), independent of the oracle's."""
    t = torch.from_numpy(np.ascontiguousarray(x32, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------ bf16 ---
def test_bf16_round_matches_library_conversion():
    r = rng(1)
    x = np.concatenate([
        r.standard_normal(20000).astype(np.float32),
        (r.standard_normal(2000) * 1e-30).astype(np.float32),
        (r.standard_normal(2000) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, np.inf, -np.inf, 3.3895314e38, 1e-45, 65504.0], dtype=np.float32),
    ])
    # exact ties (low 16 bits = 0x8000) with even and odd upper halves
    ties = (np.arange(0x3F80, 0x3F90, dtype=np.uint32) << 16 | 0x8000).view(np.float32)
    x = np.concatenate([x, ties, -ties])
    assert np.array_equal(O.bf16_round(x), torch_bf16_bits(x))
    assert O.bf16_round(np.array([np.nan], dtype=np.float32))[0] & 0x7F80 == 0x7F80


def test_bf16_to_f32_is_exact_inverse_on_bf16_values():
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)
    back = O.bf16_round(O.bf16_to_f32(bits))
    assert np.array_equal(bits, back)
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(t, O.bf16_to_f32(bits))


def test_bf16_hand_worked_values():
    # 0.6 = 1.2 * 2^-1 -> mantissa 0.2*128 = 25.6 -> 26 -> 0x3F1A (0.6015625)
    # 0.8 = 1.6 * 2^-1 -> mantissa 0.6*128 = 76.8 -> 77 -> 0x3F4D (0.80078125)
    got = O.bf16_round(np.array([0.6, 0.8, 1.0, -2.0, 0.1], dtype=np.float32))
    assert [hex(int(v)) for v in got] == ["0x3f1a", "0x3f4d", "0x3f80", "0xc000", "0x3dcd"]
    assert O.bf16_to_f32(np.array([0x3F1A, 0x3F4D], dtype=np.uint16)).tolist() == [0.6015625, 0.80078125]


# ----------------------------------------------------------- fingerprint ---
def test_pool_constant_rows_closed_form():
    v = rng(2).standard_normal(24).astype(np.float32)
    h = np.broadcast_to(v, (3, 16, 24)).copy()
    p = O.pool(h, "f32")
    assert np.array_equal(p, np.broadcast_to(v.astype(np.float64), (3, 24)))


def test_pool_exact_rational_brute_force():
    r = rng(3)
    B, n, d = 2, 5, 4
    h = r.standard_normal((B, n, d)).astype(np.float32)
    p = O.pool(h, "f32")
    for b in range(B):
        for i in range(d):
            exact = sum(Fraction(float(h[b, t, i])) for t in range(n)) / n
            assert abs(Fraction(float(p[b, i])) - exact) <= abs(exact) * Fraction(1, 10 ** 14) + Fraction(1, 10 ** 300)


def test_pool_bf16_input_reads_the_stored_values():
    r = rng(4)
    x = r.standard_normal((2, 8, 16)).astype(np.float32)
    bits = torch_bf16_bits(x)
    vals = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.allclose(O.pool(bits, "bf16"), vals.mean(axis=1), rtol=0, atol=1e-15)


def test_pool_is_invariant_to_position_order_and_not_to_feature_order():
    r = rng(5)
    h = r.standard_normal((2, 32, 8)).astype(np.float32)
    perm = r.permutation(32)
    assert np.allclose(O.pool(h, "f32"), O.pool(h[:, perm, :], "f32"), rtol=0, atol=1e-14)
    # the mean is over positions (axis 1), not over features
    h2 = np.zeros((1, 4, 3), dtype=np.float32)
    h2[0, :, 0] = [1, 2, 3, 6]
    assert O.pool(h2, "f32").tolist() == [[3.0, 0.0, 0.0]]


def test_project_one_hot_selects_and_centres():
    r = rng(6)
    p = r.standard_normal((3, 8))
    P = np.zeros((8, 2), dtype=np.float32)
    P[5, 0] = 1.0
    P[2, 1] = 1.0
    mu = r.standard_normal(8).astype(np.float32)
    g = O.project(p, torch_bf16_bits(P), mu)
    assert np.allclose(g[:, 0], p[:, 5] - mu[5].astype(np.float64), atol=1e-15)
    assert np.allclose(g[:, 1], p[:, 2] - mu[2].astype(np.float64), atol=1e-15)
    assert np.array_equal(O.project(p, None, None), p)


def test_project_exact_rational_brute_force_and_orientation():
    r = rng(7)
    d, k = 5, 3
    p = r.standard_normal((2, d))
    Pbits = torch_bf16_bits(r.standard_normal((d, k)).astype(np.float32))
    Pv = O.bf16_to_f32(Pbits)
    mu = r.standard_normal(d).astype(np.float32)
    g = O.project(p, Pbits, mu)
    for b in range(2):
        for c in range(k):
            exact = sum((Fraction(float(p[b, i])) - Fraction(float(mu[i]))) * Fraction(float(Pv[i, c]))
                        for i in range(d))
            assert abs(float(exact) - g[b, c]) < 1e-13


def test_normalise_hand_worked_3_4_5():
    q, rq = O.normalise(np.array([[3.0, 4.0]]))
    assert q.tolist() == [[0x3F1A, 0x3F4D]]
    # norm of the rounded vector: 0.6015625^2 + 0.80078125^2 = 1.0031280517578125
    assert abs(float(rq[0]) - 1.0 / math.sqrt(1.0031280517578125)) < 6e-8
    with open(os.path.join(GOLDEN, "normalise_3_4.txt")) as f:
        vals = [ln.split("#")[0].strip() for ln in f if ln.split("#")[0].strip()]
    assert [int(vals[0], 16), int(vals[1], 16)] == q[0].tolist()
    assert abs(float(rq[0]) - float(vals[2])) < 6e-8


def test_normalise_unit_norm_scale_invariance_and_degenerate():
    r = rng(8)
    g = r.standard_normal((16, 64))
    q, rq = O.normalise(g)
    qn = np.sqrt((O.bf16_to_f32(q).astype(np.float64) ** 2).sum(axis=1))
    assert np.all(np.abs(qn * rq - 1.0) < 1e-6)
    assert np.all(np.abs(qn - 1.0) < 4e-3)
    q2, rq2 = O.normalise(g * 1024.0)          # power of two: exactly the same
    assert np.array_equal(q, q2) and np.array_equal(rq, rq2)
    q3, _ = O.normalise(g * 3.7)               # any positive scale: within 1 ulp
    d = np.abs(q.astype(np.int32) - q3.astype(np.int32))
    assert d.max() <= 1 and (d != 0).mean() < 0.01
    qn_, rqn = O.normalise(-g)                  # sign matters
    assert np.array_equal(qn_, q ^ np.uint16(0x8000)) and np.array_equal(rqn, rq)
    bad = np.zeros((3, 8))
    bad[1, 2] = np.nan
    bad[2, 3] = np.inf
    qb, rqb = O.normalise(bad)
    assert not qb.any() and not rqb.any()


def test_inv_norm_of_stored():
    bits = torch_bf16_bits(np.array([[3.0, 4.0], [0.0, 0.0]], dtype=np.float32))
    rq = O.inv_norm_of_stored(bits)
    assert rq.tolist() == [np.float32(0.2), 0.0]


# ----------------------------------------------------------------- score ---
def _unit_bank(r, N, k):
    g = r.standard_normal((N, k))
    q, rq = O.normalise(g)
    return g, q, rq


def test_score_identity_is_one():
    r = rng(10)
    _, q, rq = _unit_bank(r, 32, 96)
    s = O.scores(q, rq, q, rq, np.ones(32, np.uint8))
    assert np.all(np.abs(np.diag(s) - 1.0) < 1e-6)
    best, slot, _ = O.best_match(s)
    assert slot.tolist() == list(range(32))


def test_score_matches_library_cosine_on_stored_values():
    r = rng(11)
    _, q, rq = _unit_bank(r, 20, 48)
    _, f, rb = _unit_bank(r, 37, 48)
    s = O.scores(q, rq, f, rb, np.ones(37, np.uint8))
    ref = 1.0 - cdist(O.bf16_to_f32(q).astype(np.float64), O.bf16_to_f32(f).astype(np.float64), metric="cosine")
    assert np.allclose(s, ref, rtol=0, atol=2e-7)
    # orientation: s[b, j] is query b against key j
    assert abs(s[3, 30] - ref[3, 30]) < 2e-7 and abs(ref[3, 30] - ref[30 % 20, 3]) > 1e-4


def test_score_close_to_cosine_of_unrounded_vectors():
    r = rng(12)
    g, q, rq = _unit_bank(r, 12, 256)
    s = O.scores(q, rq, q, rq, np.ones(12, np.uint8)).astype(np.float64)
    for a in range(12):
        for b in range(12):
            da = [float(x) for x in g[a]]
            db = [float(x) for x in g[b]]
            dot = math.fsum(x * y for x, y in zip(da, db))
            ref = dot / math.sqrt(math.fsum(x * x for x in da) * math.fsum(y * y for y in db))
            assert abs(s[a, b] - ref) < 1e-3
            assert abs(s[a, b] - s[b, a]) < 1e-7
            assert abs(s[a, b]) <= 1.0 + 1e-6


def test_score_orthogonal_antipodal_and_free_slots():
    k = 8
    e = np.eye(k)
    q, rq = O.normalise(e[:3])
    f, rb = O.normalise(np.stack([e[0], -e[1], e[5], e[2]]))
    valid = np.array([1, 1, 1, 0], np.uint8)
    s = O.scores(q, rq, f, rb, valid)
    assert s[0].tolist() == [1.0, 0.0, 0.0, -np.inf]
    assert s[1].tolist() == [0.0, -1.0, 0.0, -np.inf]
    assert s[2, 3] == -np.inf                       # would be 1.0 if the slot were occupied


def test_score_expected_cosine_of_perturbed_copies():
    # a copy perturbed by sigma_q of an entry built as unit-variance centre plus
    # sigma_e noise has cosine sqrt((1+se^2)/(1+se^2+sq^2)) in expectation
    r = rng(13)
    k, se, sq = 768, 0.05, 0.05
    centre = r.standard_normal((1, k))
    entry = centre + se * r.standard_normal((200, k))
    query = entry + sq * r.standard_normal((200, k))
    f, rb = O.normalise(entry)
    q, rq = O.normalise(query)
    s = O.scores(q, rq, f, rb, np.ones(200, np.uint8))
    own = np.diag(s).astype(np.float64)
    expect = math.sqrt((1 + se * se) / (1 + se * se + sq * sq))
    assert abs(expect - 0.99875) < 1e-5
    assert abs(own.mean() - expect) < 2e-4
    sib = (s.sum() - own.sum()) / (200 * 199)
    assert abs(sib - 1.0 / math.sqrt((1 + se * se + sq * sq) * (1 + se * se))) < 5e-4


# ----------------------------------------------------- argmax, threshold ---
def test_best_match_brute_force_and_ties():
    r = rng(14)
    s = r.standard_normal((9, 17)).astype(np.float32)
    s[2, 4] = s[2, 11] = 9.0          # exact tie -> lowest slot
    s[5, :] = -np.inf                 # nothing occupied
    best, slot, second = O.best_match(s)
    for b in range(9):
        bj, bv = -1, -math.inf
        for j in range(17):
            if s[b, j] > bv:
                bj, bv = j, float(s[b, j])
        assert slot[b] == bj and (best[b] == bv)
        others = [float(s[b, j]) for j in range(17) if j != bj]
        assert second[b] == (max(others) if bj >= 0 else -math.inf)
    assert slot[2] == 4 and second[2] == 9.0 and slot[5] == -1


def test_decide_strict_and_ge_on_exact_threshold():
    best = np.array([1.0, 0.95, 0.9, 0.5, -np.inf], np.float32)
    slot = np.array([3, 1, 2, 0, -1], np.int32)
    rq = np.array([1, 1, 1, 1, 1], np.float32)
    hit, out = O.decide(best, slot, rq, 0.9)
    # 0.9 as float32 equals float32(0.9): strict '>' misses, '>=' hits
    assert hit.tolist() == [1, 1, 0, 0, 0] and out.tolist() == [3, 1, -1, -1, -1]
    hit, out = O.decide(best, slot, rq, 0.9, cmp_ge=True)
    assert hit.tolist() == [1, 1, 1, 0, 0]
    hit, _ = O.decide(best, slot, rq, 1.0)
    assert hit.tolist() == [0, 0, 0, 0, 0]          # tau >= 1 under '>' : all miss
    hit, _ = O.decide(best, slot, np.array([0, 1, 1, 1, 1], np.float32), 0.0)
    assert hit.tolist() == [0, 1, 1, 1, 0]          # degenerate query never hits


def test_decide_monotone_in_tau():
    r = rng(15)
    best = r.uniform(-1, 1, 500).astype(np.float32)
    slot = np.zeros(500, np.int32)
    rq = np.ones(500, np.float32)
    prev = None
    for tau in [0.0, 0.5, 0.8, 0.82, 0.88, 0.9, 0.95, 0.999]:
        hit, _ = O.decide(best, slot, rq, tau)
        if prev is not None:
            assert np.all(hit <= prev)
        prev = hit


def test_compact_is_an_ordered_partition():
    r = rng(16)
    hit = (r.uniform(size=300) < 0.4).astype(np.uint8)
    hi, mi = O.compact(hit)
    assert sorted(hi.tolist() + mi.tolist()) == list(range(300))
    assert np.all(np.diff(hi) > 0) and np.all(np.diff(mi) > 0)
    assert all(hit[i] for i in hi) and not any(hit[i] for i in mi)
    hi, mi = O.compact(np.zeros(0, np.uint8))
    assert len(hi) == 0 and len(mi) == 0


# ----------------------------------------- whole probe / commit round trip ---
def _mk_bank(N=8, n=4, d=16, k=16, **kw):
    return O.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, **kw)


def _rand_h(r, B, n, d):
    return r.standard_normal((B, n, d)).astype(np.float32)


def _rand_act(r, M, n, d):
    return r.integers(0, 0x7F00, size=(M, n * d), dtype=np.uint16)


def test_empty_bank_all_miss_then_identity_hits_and_verbatim_reuse():
    r = rng(20)
    bank = _mk_bank()
    h = _rand_h(r, 5, 4, 16)
    pr = O.probe(bank, h, "f32")
    assert pr.hit.tolist() == [0] * 5 and np.all(pr.score == -np.inf) and pr.slot.tolist() == [-1] * 5
    out = _rand_act(r, 5, 4, 16)
    h_out = np.zeros((5, 64), np.uint16)
    new = O.commit(bank, pr, out, h_out)
    assert new.tolist() == [0, 1, 2, 3, 4] and np.array_equal(h_out, out)
    # Algorithm 1: the same input now finds its own key with sim = 1 and reuses h' verbatim
    for tau in (0.0, 0.9, 0.999):
        h_out2 = np.zeros((5, 64), np.uint16)
        pr2 = O.probe(bank, h, "f32", tau=tau, h_out=h_out2)
        assert pr2.hit.tolist() == [1] * 5 and pr2.slot.tolist() == [0, 1, 2, 3, 4]
        assert np.all(np.abs(pr2.score - 1.0) < 1e-6)
        assert np.array_equal(h_out2, out)
    pr3 = O.probe(bank, h, "f32", tau=1.0 + 1e-5)
    assert pr3.hit.sum() == 0                       # a cosine cannot exceed 1 by more than rounding


def test_snapshot_semantics_duplicates_in_one_batch_both_insert():
    r = rng(21)
    bank = _mk_bank()
    h = _rand_h(r, 1, 4, 16)
    hh = np.concatenate([h, h])
    pr = O.probe(bank, hh, "f32")
    assert pr.hit.tolist() == [0, 0]
    O.commit(bank, pr, _rand_act(r, 2, 4, 16))
    assert bank.valid.sum() == 2
    pr = O.probe(bank, h, "f32")
    assert pr.slot.tolist() == [0]                  # tie between the two copies -> lowest slot


def test_banks_of_different_layers_are_independent():
    r = rng(22)
    a, b = _mk_bank(), _mk_bank()
    h = _rand_h(r, 3, 4, 16)
    O.commit(a, O.probe(a, h, "f32"), _rand_act(r, 3, 4, 16))
    assert b.valid.sum() == 0 and b.tick == 0
    assert O.probe(b, h, "f32").hit.sum() == 0 and O.probe(a, h, "f32").hit.sum() == 3


def test_probe_brute_force_tiny_bank():
    r = rng(23)
    N, k = 6, 16
    bank = _mk_bank(N=N, n=2, d=k, k=k)
    base = _rand_h(r, N, 2, k)
    O.commit(bank, O.probe(bank, base, "f32"), _rand_act(r, N, 2, k))
    q = base[[4, 1]] + 0.1 * _rand_h(r, 2, 2, k)
    q = np.concatenate([q, _rand_h(r, 3, 2, k)])
    pr = O.probe(bank, q, "f32", tau=0.8, keep_scores=True)
    pooled = q.astype(np.float64).mean(axis=1)
    keys = base.astype(np.float64).mean(axis=1)
    for b in range(5):
        cos = [float(pooled[b] @ keys[j] / (np.linalg.norm(pooled[b]) * np.linalg.norm(keys[j]))) for j in range(N)]
        j = int(np.argmax(cos))
        assert abs(pr.score[b] - cos[j]) < 1e-3 and pr.best_slot[b] == j
        assert bool(pr.hit[b]) == (cos[j] > 0.8)
    assert pr.slot[0] == 4 and pr.slot[1] == 1


def test_degenerate_query_misses_and_is_not_inserted():
    r = rng(24)
    bank = _mk_bank()
    h = _rand_h(r, 3, 4, 16)
    h[1] = 0.0
    pr = O.probe(bank, h, "f32")
    new = O.commit(bank, pr, _rand_act(r, 3, 4, 16))
    assert new.tolist() == [0, -1, 1] and bank.valid.sum() == 2
    pr = O.probe(bank, h, "f32", tau=-0.5)
    assert pr.hit.tolist() == [1, 0, 1] and pr.score[1] == 0.0 and pr.best_slot[1] == -1


# ------------------------------------------------------ insert / eviction ---
def test_more_misses_than_slots_first_n_insert():
    r = rng(30)
    bank = _mk_bank(N=4)
    h = _rand_h(r, 7, 4, 16)
    pr = O.probe(bank, h, "f32")
    new = O.commit(bank, pr, _rand_act(r, 7, 4, 16))
    assert new.tolist() == [0, 1, 2, 3, -1, -1, -1] and bank.valid.sum() == 4


def test_lru_policy_equals_textbook_lru_list():
    r = rng(31)
    N = 5
    bank = _mk_bank(N=N, policy=O.POLICY_LRU)
    universe = _rand_h(r, 12, 4, 16)
    lru = collections.OrderedDict()          # item -> slot, oldest first
    free = list(range(N))
    for step in range(200):
        item = int(r.integers(0, 12))
        pr = O.probe(bank, universe[item:item + 1], "f32")
        if item in lru:
            assert pr.hit[0] == 1 and pr.slot[0] == lru[item]
            lru.move_to_end(item)
        else:
            assert pr.hit[0] == 0
            new = O.commit(bank, pr, _rand_act(r, 1, 4, 16))
            if free:
                slot = free.pop(0)
            else:
                _, slot = lru.popitem(last=False)
            assert new[0] == slot
            lru[item] = slot
        assert bank.valid.sum() <= N


def test_victim_has_minimal_key_independent_quadratic_scan():
    r = rng(32)
    N = 24
    bank = _mk_bank(N=N)
    universe = _rand_h(r, 60, 4, 16)
    for step in range(120):
        ids = r.integers(0, 60, size=int(r.integers(1, 6)))
        ids = np.unique(ids)
        pr = O.probe(bank, universe[ids], "f32")
        # snapshot of metadata before the commit, key recomputed here with float math
        t, e = bank.tick, bank.tick // bank.half_life_ticks
        def key(j):
            m_eff = int(math.floor(int(bank.m[j]) / 2.0 ** min(31, e - int(bank.e_upd[j]))))
            stale = m_eff < bank.stale_floor_q8 and (t - int(bank.insert_tick[j])) >= bank.min_age_ticks
            return (0 if stale else 1, m_eff, int(bank.last_use[j]), j)
        occupied = [j for j in range(N) if bank.valid[j]]
        freeb = [j for j in range(N) if not bank.valid[j]]
        keys = {j: key(j) for j in occupied}
        new = O.commit(bank, pr, _rand_act(r, len(pr.miss_idx), 4, 16))
        taken = [int(v) for v in new if v >= 0]
        assert len(set(taken)) == len(taken)
        n_free = min(len(freeb), len(taken))
        assert taken[:n_free] == freeb[:n_free]                 # free slots first, ascending
        evicted = taken[n_free:]
        for a, v in enumerate(evicted):
            assert all(keys[v] < keys[w] for w in occupied if w not in evicted[:a + 1])
        assert bank.valid.sum() <= N


def test_touch_is_order_independent_and_counts_multiplicity():
    r = rng(33)
    base = _rand_h(r, 6, 4, 16)
    acts = _rand_act(r, 6, 4, 16)
    batch = base[[0, 0, 3, 5, 3, 0]]
    states = []
    for perm in (np.arange(6), r.permutation(6), r.permutation(6)):
        bank = _mk_bank()
        O.commit(bank, O.probe(bank, base, "f32"), acts)
        pr = O.probe(bank, batch[perm], "f32")
        assert pr.hit.sum() == 6
        states.append((bank.m.copy(), bank.hits.copy(), bank.last_use.copy(), bank.e_upd.copy()))
    for s in states[1:]:
        assert all(np.array_equal(a, b) for a, b in zip(states[0], s))
    m, hits, last_use, _ = states[0]
    assert hits.tolist()[:6] == [3, 0, 0, 2, 0, 1]
    assert m.tolist()[:6] == [256 + 768, 256, 256, 256 + 512, 256, 256 + 256]
    assert last_use.tolist()[:6] == [2, 1, 1, 2, 1, 2]


def test_decayed_rate_halves_per_half_life_hand_worked():
    r = rng(34)
    bank = _mk_bank(N=4, half_life_ticks=8, stale_floor_q8=64, min_age_ticks=4)
    h = _rand_h(r, 1, 4, 16)
    other = _rand_h(r, 1, 4, 16)
    O.commit(bank, O.probe(bank, h, "f32"), _rand_act(r, 1, 4, 16))       # tick 1, epoch 0, m = 256
    assert (bank.m[0], bank.e_upd[0], bank.insert_tick[0]) == (256, 0, 1)
    while bank.tick < 23:
        O.probe(bank, other, "f32")
    assert O.effective_rate(bank, 0) == 64 and not O.is_stale(bank, 0)     # epoch 2: 256 >> 2
    O.probe(bank, other, "f32")                                            # tick 24, epoch 3: 32 < 64
    assert O.effective_rate(bank, 0) == 32 and O.is_stale(bank, 0)
    pr = O.probe(bank, h, "f32")                                           # tick 25: a hit refreshes it
    assert pr.hit[0] == 1 and bank.m[0] == 32 + 256 and bank.e_upd[0] == 3 and not O.is_stale(bank, 0)


def test_stale_entries_go_before_recently_used_ones_and_flushes():
    r = rng(35)
    bank = _mk_bank(N=4)
    items = _rand_h(r, 4, 4, 16)
    O.commit(bank, O.probe(bank, items, "f32"), _rand_act(r, 4, 4, 16))    # tick 1
    while bank.tick < 30:
        O.probe(bank, items[[1, 3]], "f32")                                # 1 and 3 stay hot
    assert [O.is_stale(bank, j) for j in range(4)] == [True, False, True, False]
    assert O.victim_order(bank) == [0, 2, 1, 3]
    lru_bank = _mk_bank(N=4, policy=O.POLICY_LRU)
    assert not O.is_stale(lru_bank, 0)
    import copy
    b2 = copy.deepcopy(bank)
    assert O.evict(b2, O.EVICT_STALE) == 2 and b2.valid.tolist() == [0, 1, 0, 1]
    b3 = copy.deepcopy(bank)
    b3.max_idle_ticks = 10
    assert O.evict(b3, O.EVICT_IDLE) == 2 and b3.valid.tolist() == [0, 1, 0, 1]
    b3.max_idle_ticks = 29
    assert O.evict(b3, O.EVICT_IDLE) == 0
    b4 = copy.deepcopy(bank)
    assert O.evict(b4, O.EVICT_SLOTS, [1, 2]) == 2 and b4.valid.tolist() == [1, 0, 0, 1]
    assert O.evict(b4, O.EVICT_ALL) == 2 and b4.valid.sum() == 0
    new = O.commit(bank, O.probe(bank, _rand_h(r, 3, 4, 16), "f32"), _rand_act(r, 3, 4, 16))
    assert new.tolist() == [0, 2, 1]


def test_churn_junk_is_evicted_before_regularly_hit_entries():
    r = rng(36)
    N = 32
    bank = _mk_bank(N=N)
    live = _rand_h(r, 8, 4, 16)
    O.commit(bank, O.probe(bank, live, "f32"), _rand_act(r, 8, 4, 16))
    live_slots = set(range(8))
    for step in range(60):
        junk = _rand_h(r, 6, 4, 16)
        batch = np.concatenate([live, junk])
        pr = O.probe(bank, batch, "f32", tau=0.9)
        assert pr.hit[:8].sum() == 8 and pr.hit[8:].sum() == 0
        new = O.commit(bank, pr, _rand_act(r, 6, 4, 16))
        assert not (set(int(v) for v in new) & live_slots)
        assert bank.valid.sum() <= N


def test_act_rows_aliasing_maps_slot_modulo():
    r = rng(37)
    bank = _mk_bank(N=8, act_rows=4)
    h = _rand_h(r, 6, 4, 16)
    acts = _rand_act(r, 6, 4, 16)
    O.commit(bank, O.probe(bank, h, "f32"), acts)
    h_out = np.zeros((6, 64), np.uint16)
    pr = O.probe(bank, h, "f32", h_out=h_out)
    assert pr.slot.tolist() == list(range(6))
    assert np.array_equal(h_out[5], acts[5]) and np.array_equal(h_out[1], acts[5])   # rows 1 and 5 share storage


# --------------------------------------------------------------------------------- SimHash ---
def test_simhash_bits_hamming_brute_force_and_threshold():
    r = rng(40)
    g = r.standard_normal((6, 64))
    q, rq = O.normalise(g)
    bits_ = O.simhash_bits(q)
    assert np.array_equal(bits_, (g < 0).astype(np.uint8))                 # sign of the projection
    assert O.hamming_threshold(1.0, 256) == -1 and O.hamming_threshold(-1.0, 256) == 256
    for tau in (0.0, 0.5, 0.82, 0.9):
        hm = O.hamming_threshold(tau, 256)
        assert math.cos(math.pi * hm / 256) > tau >= math.cos(math.pi * (hm + 1) / 256) - 1e-12
    bank = _mk_bank(N=8, n=2, d=64, k=64)
    base = _rand_h(r, 5, 2, 64)
    O.commit(bank, O.probe(bank, base, "f32"), _rand_act(r, 5, 2, 64))
    qh = base[[3, 1]] + 0.05 * _rand_h(r, 2, 2, 64)
    fq, rqq = O.fingerprint(qh, "f32")
    pr, ham = O.probe_simhash(bank, fq, rqq, tau=0.8)
    for b in range(2):
        qb = [int(x) >> 15 for x in fq[b]]
        dist = [sum(1 for c in range(64) if qb[c] != (int(bank.fp[j][c]) >> 15)) for j in range(5)]
        assert ham[b] == min(dist) and pr.best_slot[b] == dist.index(min(dist))
        assert abs(pr.score[b] - math.cos(math.pi * min(dist) / 64)) < 1e-6
    assert pr.slot.tolist() == [3, 1]
    fs, rs = O.fingerprint(base[:1], "f32")                                 # identical input: distance 0, score 1
    pr, ham = O.probe_simhash(bank, fs, rs, tau=0.99)
    assert ham[0] == 0 and pr.score[0] == 1.0 and pr.hit[0] == 1


def test_simhash_angle_estimate_is_unbiased_for_random_hyperplanes():
    # P(sign differs) = theta / pi for a random hyperplane: the mean normalised distance estimates the angle
    r = rng(41)
    d, k = 48, 4096
    a = r.standard_normal(d); b = a + 0.6 * r.standard_normal(d)
    theta = math.acos(float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b))))
    P = r.standard_normal((d, k))
    ha = O.simhash_bits(O.normalise((a @ P)[None])[0]); hb = O.simhash_bits(O.normalise((b @ P)[None])[0])
    frac = float((ha != hb).mean())
    assert abs(frac - theta / math.pi) < 4 * math.sqrt(0.25 / k)


# ------------------------------------------------ pooled probing, augmented ---
def test_probe_pooled_equals_probe_on_the_hidden_states_and_exact_means():
    # position means in exact rational arithmetic of the written layer output -> same decisions as probe()
    r = rng(77)
    B, n, d, k, N = 6, 5, 16, 64, 8
    P = O.bf16_round((r.standard_normal((d, k)) / math.sqrt(k)).astype(np.float32))
    h = O.bf16_round(r.standard_normal((B, n, d)).astype(np.float32))
    bank_a = O.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, proj=P, tau=0.5)
    bank_b = O.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, proj=P, tau=0.5)
    for bk in (bank_a, bank_b):
        pr = O.probe(bk, h[:4], "bf16")
        O.commit(bk, pr, h[:4].reshape(4, -1))
    vals = O.bf16_to_f32(h)
    means = np.array([[float(sum(Fraction(float(vals[b, t, i])) for t in range(n)) / n) for i in range(d)]
                      for b in range(B)])
    pa = O.probe(bank_a, h, "bf16")
    pb = O.probe_pooled(bank_b, means)
    assert np.array_equal(pa.fp, pb.fp) and np.array_equal(pa.hit, pb.hit) and np.array_equal(pa.slot, pb.slot)
    assert pa.hit[:4].all() and not pa.hit[4:].any()
    assert np.array_equal(pa.score, pb.score)


def test_fingerprint_augmented_block_structure():
    # a block-diagonal projection separates the two parts: each block equals the plain projection of its part
    r = rng(78)
    B, n, d, k = 4, 7, 8, 64
    h = r.standard_normal((B, n, d)).astype(np.float32)
    a = O.bf16_round(r.standard_normal((B, n, d)).astype(np.float32))
    P1 = O.bf16_round(r.standard_normal((d, k // 2)).astype(np.float32))
    P2 = O.bf16_round(r.standard_normal((d, k // 2)).astype(np.float32))
    Pfull = np.zeros((2 * d, k), dtype=np.uint16)
    Pfull[:d, :k // 2] = P1
    Pfull[d:, k // 2:] = P2
    fp, rq = O.fingerprint_augmented(h, "f32", a, "bf16", Pfull, None)
    g1 = h.astype(np.float64).mean(axis=1) @ O.bf16_to_f32(P1).astype(np.float64)
    g2 = O.bf16_to_f32(a).astype(np.float64).mean(axis=1) @ O.bf16_to_f32(P2).astype(np.float64)
    g = np.concatenate([g1, g2], axis=1)
    want = g / np.linalg.norm(g, axis=1, keepdims=True)
    got = O.bf16_to_f32(fp).astype(np.float64)
    assert np.max(np.abs(got - want)) <= 2.0 ** -8          # one bf16 rounding of values below 1
    # zeroing the attention part reduces it to the plain fingerprint with the first block
    fp0, _ = O.fingerprint_augmented(h, "f32", np.zeros_like(a), "bf16", Pfull, None)
    fpp, _ = O.fingerprint(h, "f32", np.ascontiguousarray(Pfull[:d]), None)
    assert np.array_equal(fp0, fpp)
    # swapping the two inputs is not the same fingerprint (the order of the parts matters)
    fps, _ = O.fingerprint_augmented(O.bf16_to_f32(a), "f32", O.bf16_round(h), "bf16", Pfull, None)
    assert not np.array_equal(fps, fp)
