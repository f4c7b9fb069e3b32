"""Host logic of the bank that is split over several ranks, on the CPU with two gloo ranks.

The one exchange step of a split bank is an element-wise unsigned maximum of one packed 64-bit word per query
(score in an order-preserving integer form above, inverted slot below).  Here each rank scores its slice of a
small bank with the oracle, packs its best words in the documented format, the ranks combine them with
combine_words, and the result must be the oracle's best match over the whole bank: the same slot (lowest on
equal scores) and the same score.  No kernel runs; what is checked is the word format, the exchange and the
way slots and misses are shared out.
"""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def pack_words(score_f32: np.ndarray, slot: np.ndarray) -> np.ndarray:
    """(score, slot) -> uint64 word: the float's bits made order-preserving (negative: all bits inverted;
    non-negative: top bit set), shifted up by 32, with 2^32 - 1 - slot below.  slot < 0 (no key) -> 0."""
    u = score_f32.astype(np.float32).view(np.uint32).astype(np.uint64)
    o = np.where(u >> np.uint64(31), u ^ np.uint64(0xFFFFFFFF), u | np.uint64(0x80000000))
    w = (o << np.uint64(32)) | (np.uint64(0xFFFFFFFF) - slot.astype(np.int64).clip(0).astype(np.uint64))
    return np.where(slot < 0, np.uint64(0), w)


def unpack_words(w: np.ndarray):
    o = (w >> np.uint64(32)).astype(np.uint32)
    u = np.where(o >> np.uint32(31), o & np.uint32(0x7FFFFFFF), ~o)
    return u.astype(np.uint32).view(np.float32), (np.uint64(0xFFFFFFFF) - (w & np.uint64(0xFFFFFFFF))).astype(np.int64)


def _bank_and_queries():
    sys.path.insert(0, ROOT)
    from oracle import llmcache_oracle as O
    rng = np.random.Generator(np.random.Philox(key=77))
    N, B, k = 301, 40, 64
    keys = rng.standard_normal((N, k))
    keys[150] = keys[3]                                  # an exact duplicate: the tie must go to slot 3
    keys[200] = -keys[7]                                 # an antipodal key: negative scores take part too
    fp = O.bf16_round((keys / np.linalg.norm(keys, axis=1, keepdims=True)).astype(np.float32))
    q = rng.standard_normal((B, k))
    q[:10] = keys[rng.integers(0, N, 10)] + 0.05 * rng.standard_normal((10, k))
    q[10] = keys[3]
    q[11] = -keys[5] - keys[7]                           # every score negative for some keys
    qf = O.bf16_round((q / np.linalg.norm(q, axis=1, keepdims=True)).astype(np.float32))
    valid = np.ones(N, dtype=np.uint8)
    valid[::13] = 0
    return O, fp, qf, valid


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2512_16843_b200 import sharded as S
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    O, fp, qf, valid = _bank_and_queries()
    N = fp.shape[0]
    first, count = S.slice_bounds(N, world, rank)
    sl = slice(first, first + count)
    rq = O.inv_norm_of_stored(qf)
    s = O.scores(qf, np.ones_like(rq), fp[sl], O.inv_norm_of_stored(fp[sl]), valid[sl])    # the scan leaves 1/|q| to the decision
    best, slot, _ = O.best_match(s)
    words = pack_words(best, np.where(slot >= 0, slot + first, -1))
    t = torch.from_numpy(words.view(np.int64).copy())
    S.combine_words(t)
    out.put((rank, t.numpy().view(np.uint64).copy(), first, count))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_combine_their_best_words_into_the_oracle_s_best_match():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in range(2)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert np.array_equal(res[0][1], res[1][1])                          # every rank ends with the same words
    assert (res[0][2], res[0][3], res[1][2], res[1][3]) == (0, 151, 151, 150)
    O, fp, qf, valid = _bank_and_queries()
    rq = O.inv_norm_of_stored(qf)
    s = O.scores(qf, np.ones_like(rq), fp, O.inv_norm_of_stored(fp), valid)
    best, slot, _ = O.best_match(s)
    score, got_slot = unpack_words(res[0][1])
    assert np.array_equal(got_slot, slot)
    assert np.array_equal(score.view(np.uint32), best.view(np.uint32))
    assert got_slot[10] == 3                                             # the duplicate at slot 150 loses the tie


def test_word_order_is_the_order_of_score_then_lowest_slot():
    sc = np.array([-1.0, -0.25, -0.0, 0.0, 1e-30, 0.5, 0.5, 1.0], dtype=np.float32)
    sl = np.array([5, 5, 5, 5, 5, 9, 2, 0])
    w = pack_words(sc, sl)
    assert w[0] < w[1] < w[2] < w[3] < w[4] < w[5] < w[6] < w[7]         # 0.5 at slot 2 beats 0.5 at slot 9
    assert pack_words(np.array([3.0], np.float32), np.array([-1]))[0] == 0
    back, slot = unpack_words(w)
    assert np.array_equal(back.view(np.uint32), sc.view(np.uint32)) and np.array_equal(slot, sl)
    # the signed detour of combine_words is an unsigned maximum
    sys.path.insert(0, ROOT)
    from paper_2512_16843_b200 import sharded as S
    a = torch.from_numpy(w.view(np.int64).copy())
    b = torch.from_numpy(w[::-1].copy().view(np.int64).copy())
    m = S.unsigned_max_(a.clone(), b).numpy().view(np.uint64)
    assert np.array_equal(m, np.maximum(w, w[::-1]))


def test_slots_and_misses_are_shared_out_without_gaps_or_overlaps():
    sys.path.insert(0, ROOT)
    from paper_2512_16843_b200 import sharded as S
    for n_total, world in ((1024, 4), (301, 2), (7, 3), (5, 8)):
        cover = []
        for r in range(world):
            first, count = S.slice_bounds(n_total, world, r)
            cover += list(range(first, first + count))
        assert cover == list(range(n_total))
    for M, world in ((0, 2), (1, 2), (10, 3), (65, 8)):
        got = sorted(int(x) for r in range(world) for x in S.misses_of(r, world, M))
        assert got == list(range(M))
