"""Slow, plain CPU oracle for the LLMCache per-layer cache probe.

TEST INFRASTRUCTURE ONLY.  This module is the yardstick the CUDA library is
checked against; it is imported by the tests, by the smoke check and by the
benchmark's CPU-baseline timing, and by nothing else.  It shares no code with
the CUDA path and never imports it.

What it computes follows the paper (LLMCache, "Layer-Wise Caching Strategies
for Accelerated Reuse in Transformer Inference"):

* Sec. IV-B, bullet "Embedding Aggregation": the fingerprint starts from the
  average of the [n, d] hidden-state matrix over its n positions.
* Sec. IV-B, bullet "Dimensionality Reduction": the pooled vector is projected
  to a compact fixed-length vector (a linear map; the paper names PCA/SimHash
  and gives no matrix, so the matrix and the centring vector are inputs).
* Sec. III-C and Sec. IV-B last sentence: fingerprints are compared by cosine
  similarity against every key of the layer's bank.
* Sec. IV-A (the case equation) and Algorithm 1: a key whose similarity
  exceeds tau means "reuse the stored layer output", otherwise "compute the
  layer and store the result".
* Sec. III-E and Sec. IV-D: least-recently-used eviction, and staleness-aware
  eviction driven by a match rate that decays over time.

All floating-point work is done in float64 over the exact input values; the
only places where precision is fixed are the ones the stored formats fix:
fingerprints are stored as bfloat16 (round to nearest even) and scores and
inverse norms are reported as float32.  Integer bookkeeping is exact.

Readings where the paper is silent (each one is also listed in the design
notes of the repository):

* one decision per sequence; the cached value is the whole [n, d] output;
* the best-scoring key is taken, exact ties go to the lowest slot;
* the comparison is strict (">", as in the equation and Algorithm 1) unless
  `cmp_ge` is set (">=", as in Sec. III-C);
* a fingerprint whose norm is zero or not finite never hits and is never
  inserted;
* all sequences of one probe call see the bank as it was when the call began;
* "recency" is the tick of the last hit, or of insertion if never hit;
* the decayed match rate is an integer in Q8 fixed point that is halved once
  per `half_life_ticks` probe calls (a shift), plus 256 per hit;
* eviction order: free slots in ascending order first, then occupied slots in
  ascending order of (class, decayed rate, last use, slot) where class 0 is
  "stale" (rate under `stale_floor_q8` and older than `min_age_ticks`).

Parity status: every function below is pinned by tests/test_oracle_*.py
against closed forms, brute force, textbook routines or hand-worked values.
The paper prints no worked numerical example of a fingerprint, a score or an
eviction, so no pin comes from a printed number; end-to-end latency figures of
the paper (Table I) depend on data and weights that are not available:
parity unpinned for those (they are not computed here).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

M_CAP = (1 << 30) - 1          # ceiling of the decayed match rate (Q8)
HIT_INCREMENT_Q8 = 256         # one match, in Q8
POLICY_LRU = 0
POLICY_LRU_STALENESS = 1
EVICT_STALE = 0
EVICT_IDLE = 1
EVICT_ALL = 2
EVICT_SLOTS = 3
U32_MAX = (1 << 32) - 1


# --------------------------------------------------------------------------
# bfloat16 storage format (1 sign, 8 exponent, 7 mantissa bits): conversion by
# bit manipulation, round to nearest, ties to even.
# --------------------------------------------------------------------------
def bf16_round(x) -> np.ndarray:
    """float32 values -> bfloat16 bit patterns (uint16), round-nearest-even."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    u = x32.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)
    nan = np.isnan(x32)
    if np.any(nan):
        r = np.where(nan, np.uint16(0x7FC0), r)
    return r.astype(np.uint16)


def bf16_to_f32(bits) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> the float32 values they denote."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def _as_f64(h, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return bf16_to_f32(h).astype(np.float64)
    if dtype == "f32":
        return np.asarray(h, dtype=np.float32).astype(np.float64)
    raise ValueError("dtype must be 'bf16' or 'f32'")


# --------------------------------------------------------------------------
# Fingerprint (Sec. IV-B)
# --------------------------------------------------------------------------
def pool(h, dtype: str) -> np.ndarray:
    """Embedding aggregation, Sec. IV-B bullet 1: p[b,:] = (1/n) sum_t h[b,t,:].

    h: [B, n, d] (float32 values, or uint16 bfloat16 patterns).  Returns
    float64 [B, d]."""
    B, n, d = h.shape
    p = np.empty((B, d), dtype=np.float64)
    for b in range(B):                      # one sequence at a time (memory)
        p[b] = _as_f64(h[b], dtype).sum(axis=0) / float(n)
    return p


def project(p: np.ndarray, proj_bf16: Optional[np.ndarray],
            center_f32: Optional[np.ndarray]) -> np.ndarray:
    """Dimensionality reduction, Sec. IV-B bullet 3: g = (p - mu) . P.

    proj_bf16: [d, k] bfloat16 patterns or None (identity, k = d);
    center_f32: [d] float32 or None (zero).  Returns float64 [B, k]."""
    x = p
    if center_f32 is not None:
        x = x - np.asarray(center_f32, dtype=np.float32).astype(np.float64)[None, :]
    if proj_bf16 is None:
        return np.array(x, dtype=np.float64)
    P = bf16_to_f32(proj_bf16).astype(np.float64)
    return x @ P


def normalise(g: np.ndarray):
    """Unit-length fingerprint in its stored format.

    q[b,:] = bf16(g[b,:] / ||g[b]||), rq[b] = float32(1 / ||q[b]||) with the
    norm of the *rounded* vector, so that a key compared with itself has
    cosine 1 up to float32 rounding.  Degenerate vectors (norm under 1e-20 or
    any non-finite element) give q = 0 and rq = 0.
    Returns (uint16 [B,k], float32 [B])."""
    B, k = g.shape
    q = np.zeros((B, k), dtype=np.uint16)
    rq = np.zeros((B,), dtype=np.float32)
    for b in range(B):
        row = g[b]
        if not np.all(np.isfinite(row)):
            continue
        nrm = float(np.sqrt(np.sum(row * row)))
        if not np.isfinite(nrm) or nrm < 1e-20:
            continue
        qb = bf16_round((row / nrm).astype(np.float32))
        qn = float(np.sqrt(np.sum(bf16_to_f32(qb).astype(np.float64) ** 2)))
        if qn == 0.0:
            continue
        q[b] = qb
        rq[b] = np.float32(1.0 / qn)
    return q, rq


def inv_norm_of_stored(fp_bf16: np.ndarray) -> np.ndarray:
    """rq for fingerprints handed over already in bfloat16 (precomputed keys):
    float32(1/||fp||), or 0 for a zero / non-finite row."""
    v = bf16_to_f32(fp_bf16).astype(np.float64)
    B = v.shape[0]
    rq = np.zeros((B,), dtype=np.float32)
    for b in range(B):
        if not np.all(np.isfinite(v[b])):
            continue
        nn = float(np.sqrt(np.sum(v[b] * v[b])))
        if nn < 1e-20 or not np.isfinite(nn):
            continue
        rq[b] = np.float32(1.0 / nn)
    return rq


def fingerprint(h, dtype: str, proj_bf16=None, center_f32=None):
    """Sec. IV-B: pool, project, normalise.  Returns (fp uint16 [B,k], rq f32 [B])."""
    return normalise(project(pool(h, dtype), proj_bf16, center_f32))


# --------------------------------------------------------------------------
# Bank state (Sec. III-B: one independent bank of (f, h_l) tuples per layer)
# --------------------------------------------------------------------------
@dataclass
class Bank:
    capacity: int                 # N
    seq_len: int                  # n
    d_model: int                  # d
    fp_dim: int                   # k
    act_rows: int = 0             # rows of the activation store (0 => N)
    tau: float = 0.9
    cmp_ge: bool = False
    policy: int = POLICY_LRU_STALENESS
    half_life_ticks: int = 8
    stale_floor_q8: int = 64
    min_age_ticks: int = 4
    max_idle_ticks: int = 32
    proj: Optional[np.ndarray] = None      # uint16 [d, k] or None
    center: Optional[np.ndarray] = None    # float32 [d] or None
    store_act: bool = True
    tick: int = 0
    fp: np.ndarray = field(default=None, repr=False)
    rb: np.ndarray = field(default=None, repr=False)
    valid: np.ndarray = field(default=None, repr=False)
    last_use: np.ndarray = field(default=None, repr=False)
    insert_tick: np.ndarray = field(default=None, repr=False)
    hits: np.ndarray = field(default=None, repr=False)
    m: np.ndarray = field(default=None, repr=False)
    e_upd: np.ndarray = field(default=None, repr=False)
    act: np.ndarray = field(default=None, repr=False)

    def __post_init__(self):
        N = self.capacity
        if self.act_rows == 0:
            self.act_rows = N
        if self.fp is None:
            self.fp = np.zeros((N, self.fp_dim), dtype=np.uint16)
            self.rb = np.zeros((N,), dtype=np.float32)
            self.valid = np.zeros((N,), dtype=np.uint8)
            self.last_use = np.zeros((N,), dtype=np.uint32)
            self.insert_tick = np.zeros((N,), dtype=np.uint32)
            self.hits = np.zeros((N,), dtype=np.uint32)
            self.m = np.zeros((N,), dtype=np.uint32)
            self.e_upd = np.zeros((N,), dtype=np.uint32)
        if self.act is None and self.store_act:
            self.act = np.zeros((self.act_rows, self.seq_len * self.d_model), dtype=np.uint16)

    def epoch(self, tick: Optional[int] = None) -> int:
        t = self.tick if tick is None else tick
        return t // self.half_life_ticks


# --------------------------------------------------------------------------
# Matching (Sec. III-C; Sec. IV-A case equation; Algorithm 1, the "exists" test)
# --------------------------------------------------------------------------
def scores(q_bf16, rq, bank_fp_bf16, rb, valid, chunk: int = 8192) -> np.ndarray:
    """Cosine of every query against every key, Sec. III-C / IV-B:
    s[b,j] = float32(rq[b] * rb[j] * sum_c q[b,c] * f[j,c]) for occupied j,
    -inf for a free slot.  float64 arithmetic.  Returns float32 [B, N]."""
    Q = bf16_to_f32(q_bf16).astype(np.float64)
    Q[np.asarray(rq) <= 0] = 0.0              # degenerate queries score 0 everywhere
    B = Q.shape[0]
    N = bank_fp_bf16.shape[0]
    out = np.full((B, N), -np.inf, dtype=np.float32)
    rq64 = np.asarray(rq, dtype=np.float32).astype(np.float64)
    for j0 in range(0, N, chunk):
        j1 = min(N, j0 + chunk)
        F = bf16_to_f32(bank_fp_bf16[j0:j1]).astype(np.float64)
        dots = Q @ F.T
        s = dots * rq64[:, None] * np.asarray(rb[j0:j1], dtype=np.float32).astype(np.float64)[None, :]
        s32 = s.astype(np.float32)
        ok = np.asarray(valid[j0:j1]) != 0
        out[:, j0:j1] = np.where(ok[None, :], s32, np.float32(-np.inf))
    return out


def best_match(s: np.ndarray):
    """Best key per query: (best float32 [B], slot int32 [B], second float32 [B]).

    slot = lowest index attaining the maximum (np.argmax returns the first);
    best = -inf and slot = -1 if no slot is occupied; `second` = the largest
    score at any other slot (-inf if none), used only to recognise near-ties."""
    B, N = s.shape
    best = np.full((B,), -np.inf, dtype=np.float32)
    slot = np.full((B,), -1, dtype=np.int32)
    second = np.full((B,), -np.inf, dtype=np.float32)
    if N == 0:
        return best, slot, second
    for b in range(B):
        row = s[b]
        j = int(np.argmax(row))
        if row[j] == -np.inf:
            continue
        best[b] = row[j]
        slot[b] = j
        if N > 1:
            second[b] = max(np.max(row[:j], initial=-np.inf), np.max(row[j + 1:], initial=-np.inf))
    return best, slot, second


def decide(best, slot, rq, tau: float, cmp_ge: bool = False):
    """Sec. IV-A case equation / Algorithm 1: hit iff sim > tau (or >= tau,
    Sec. III-C, when cmp_ge).  The comparison is made in float32.  A degenerate
    query (rq == 0) never hits.  Misses get slot -1.
    Returns (hit uint8 [B], slot int32 [B])."""
    t32 = np.float32(tau)
    b32 = np.asarray(best, dtype=np.float32)
    over = (b32 >= t32) if cmp_ge else (b32 > t32)
    hit = over & (np.asarray(rq) > 0) & (np.asarray(slot) >= 0)
    out_slot = np.where(hit, slot, -1).astype(np.int32)
    return hit.astype(np.uint8), out_slot


def compact(hit):
    """Indices of hits and of misses, each ascending.  Returns (hit_idx, miss_idx) int32."""
    hit = np.asarray(hit)
    idx = np.arange(hit.shape[0], dtype=np.int32)
    return idx[hit != 0].copy(), idx[hit == 0].copy()


# --------------------------------------------------------------------------
# One probe call (Algorithm 1, the lookup and the reuse branch, for a batch)
# --------------------------------------------------------------------------
@dataclass
class ProbeResult:
    fp: np.ndarray          # uint16 [B,k] query fingerprints
    rq: np.ndarray          # float32 [B]
    score: np.ndarray       # float32 [B] best cosine (-inf if bank empty; 0 if rq == 0)
    second: np.ndarray      # float32 [B]
    best_slot: np.ndarray   # int32 [B] argmax before thresholding (-1 if none)
    hit: np.ndarray         # uint8 [B]
    slot: np.ndarray        # int32 [B] (-1 on miss)
    hit_idx: np.ndarray
    miss_idx: np.ndarray
    tick: int
    all_scores: Optional[np.ndarray] = None


def touch(bank: Bank, hit_slots: np.ndarray) -> None:
    """Refresh metadata of matched entries (Sec. III-E / IV-D: recency for LRU,
    match frequency, decayed match rate).  Order-independent: a slot matched
    by c queries in this call gets one decay step and +256*c."""
    t = bank.tick
    e = bank.epoch()
    if len(hit_slots) == 0:
        return
    uniq, counts = np.unique(np.asarray(hit_slots, dtype=np.int64), return_counts=True)
    for j, c in zip(uniq.tolist(), counts.tolist()):
        shift = min(31, e - int(bank.e_upd[j]))
        decayed = int(bank.m[j]) >> shift
        bank.m[j] = min(M_CAP, decayed + HIT_INCREMENT_Q8 * c)
        bank.e_upd[j] = e
        bank.last_use[j] = t
        bank.hits[j] = min(U32_MAX, int(bank.hits[j]) + c)


def probe_fp(bank: Bank, q_bf16, rq, tau: Optional[float] = None,
             h_out: Optional[np.ndarray] = None, keep_scores: bool = False) -> ProbeResult:
    """Probe with given query fingerprints.  Advances the bank's tick, finds the
    best key per query, thresholds, compacts, copies stored outputs of hits
    into h_out[b] (verbatim: Algorithm 1 "h_l <- h'"), refreshes metadata."""
    bank.tick += 1
    tau = bank.tau if tau is None else tau
    s = scores(q_bf16, rq, bank.fp, bank.rb, bank.valid)
    best, bslot, second = best_match(s)
    degenerate = np.asarray(rq) <= 0          # reported as score 0, no slot
    best[degenerate] = np.float32(0.0)
    bslot[degenerate] = -1
    second[degenerate] = np.float32(-np.inf)
    hit, slot = decide(best, bslot, rq, tau, bank.cmp_ge)
    hit_idx, miss_idx = compact(hit)
    if h_out is not None and bank.act is not None:
        for b in hit_idx.tolist():
            h_out[b] = bank.act[int(slot[b]) % bank.act_rows]
    touch(bank, slot[hit_idx])
    return ProbeResult(fp=q_bf16, rq=rq, score=best, second=second, best_slot=bslot,
                       hit=hit, slot=slot, hit_idx=hit_idx, miss_idx=miss_idx,
                       tick=bank.tick, all_scores=s if keep_scores else None)


def probe(bank: Bank, h, dtype: str, tau: Optional[float] = None,
          h_out: Optional[np.ndarray] = None, keep_scores: bool = False) -> ProbeResult:
    """Probe with the layer's input hidden states h [B, n, d]."""
    q, rq = fingerprint(h, dtype, bank.proj, bank.center)
    return probe_fp(bank, q, rq, tau, h_out, keep_scores)


def probe_pooled(bank: Bank, p, tau: Optional[float] = None,
                 h_out: Optional[np.ndarray] = None, keep_scores: bool = False) -> ProbeResult:
    """Probe when the embedding aggregation (Sec. IV-B bullet 1) of the layer's
    input is already at hand: p [B, d] are the position means.  A layer's input
    is the previous layer's output, so p can be taken while that output is
    written; the result is by definition that of probe() on the same hidden
    states."""
    q, rq = normalise(project(np.asarray(p, dtype=np.float64), bank.proj, bank.center))
    return probe_fp(bank, q, rq, tau, h_out, keep_scores)


def fingerprint_augmented(h, dtype: str, attn, attn_dtype: str, proj_bf16=None, center_f32=None):
    """Sec. IV-B with the optional second bullet ("Prefix Attention Stats": the
    fingerprint may also draw on the initial self-attention outputs): the
    position mean of the first layer's self-attention output attn [B, n, d] is
    appended to the position mean of the embeddings h [B, n, d]; the 2d-wide
    vector is then projected (proj [2d, k], center [2d]) and normalised like any
    other.  How the two parts are combined is not given in the paper;
    concatenation before the projection is the reading taken here.
    Returns (fp uint16 [B,k], rq f32 [B])."""
    p = np.concatenate([pool(h, dtype), pool(attn, attn_dtype)], axis=1)
    return normalise(project(p, proj_bf16, center_f32))


# --------------------------------------------------------------------------
# Insert on miss and eviction (Algorithm 1 "C_l[f_X] <- h_l"; Sec. III-E, IV-D)
# --------------------------------------------------------------------------
def effective_rate(bank: Bank, j: int) -> int:
    """Decayed match rate of slot j as of the bank's current tick."""
    return int(bank.m[j]) >> min(31, bank.epoch() - int(bank.e_upd[j]))


def is_stale(bank: Bank, j: int) -> bool:
    """Staleness class (Sec. IV-D: the staleness signal is a match rate that decays with time)."""
    return (bank.policy == POLICY_LRU_STALENESS
            and effective_rate(bank, j) < bank.stale_floor_q8
            and bank.tick - int(bank.insert_tick[j]) >= bank.min_age_ticks)


def eviction_key(bank: Bank, j: int):
    """Sort key of an occupied slot; smaller = evicted earlier."""
    if bank.policy == POLICY_LRU:
        return (0, 0, int(bank.last_use[j]), j)
    cls = 0 if is_stale(bank, j) else 1
    return (cls, effective_rate(bank, j), int(bank.last_use[j]), j)


def victim_order(bank: Bank):
    """All slots in the order they would be taken: free ascending, then
    occupied by ascending key."""
    free = [j for j in range(bank.capacity) if not bank.valid[j]]
    occ = sorted((j for j in range(bank.capacity) if bank.valid[j]),
                 key=lambda j: eviction_key(bank, j))
    return free + occ


def commit(bank: Bank, pr: ProbeResult, miss_out: Optional[np.ndarray],
           h_out: Optional[np.ndarray] = None) -> np.ndarray:
    """After the layer ran on the misses: scatter their outputs to h_out and
    insert them (Algorithm 1 else-branch).  miss_out: [M, n*d] uint16 in the
    order of pr.miss_idx.  Misses with rq == 0 are not inserted; the i-th
    insertable miss takes the i-th slot of the victim order; insertable misses
    beyond the capacity are dropped.  Returns new_slot int32 [M] (-1 = dropped)."""
    M = len(pr.miss_idx)
    new_slot = np.full((M,), -1, dtype=np.int32)
    insertable = [m for m in range(M) if pr.rq[int(pr.miss_idx[m])] > 0]
    take = min(len(insertable), bank.capacity)
    order = victim_order(bank)[:take]
    t = bank.tick
    e = bank.epoch()
    for i in range(take):
        m = insertable[i]
        v = order[i]
        b = int(pr.miss_idx[m])
        new_slot[m] = v
        bank.fp[v] = pr.fp[b]
        bank.rb[v] = pr.rq[b]
        bank.valid[v] = 1
        bank.last_use[v] = t
        bank.insert_tick[v] = t
        bank.hits[v] = 0
        bank.m[v] = HIT_INCREMENT_Q8
        bank.e_upd[v] = e
        if bank.act is not None and miss_out is not None:
            bank.act[v % bank.act_rows] = miss_out[m]
    if h_out is not None and miss_out is not None:
        for m in range(M):
            h_out[int(pr.miss_idx[m])] = miss_out[m]
    return new_slot


def evict(bank: Bank, mode: int, slots=None) -> int:
    """Refresh controller flush (Sec. III-E, time-based decay: entries that have gone unused or
    unmatched for too long are dropped).  Returns the number of entries removed."""
    removed = 0
    for j in range(bank.capacity):
        if not bank.valid[j]:
            continue
        if mode == EVICT_STALE:
            go = is_stale(bank, j)
        elif mode == EVICT_IDLE:
            go = bank.tick - int(bank.last_use[j]) > bank.max_idle_ticks
        elif mode == EVICT_ALL:
            go = True
        elif mode == EVICT_SLOTS:
            go = slots is not None and j in set(int(x) for x in slots)
        else:
            raise ValueError("unknown eviction mode")
        if go:
            bank.valid[j] = 0
            removed += 1
    return removed


# --------------------------------------------------------------------------
# SimHash fingerprints (named in Sec. III-A among the hashing techniques and in Sec. IV-B as one of the two
# ways to shorten the pooled vector)
# --------------------------------------------------------------------------
def simhash_bits(fp_bf16: np.ndarray) -> np.ndarray:
    """k-bit code of a fingerprint: bit c = sign bit of the projected component c (random-hyperplane
    SimHash: the projection matrix is the hyperplane matrix).  The stored bf16 fingerprint is a positive
    multiple of the projection, so its sign bits are the code.  Returns uint8 [B, k] of 0/1."""
    return ((np.asarray(fp_bf16, dtype=np.uint16) >> 15) & 1).astype(np.uint8)


def hamming_threshold(tau: float, k: int) -> int:
    """Largest Hamming distance that still counts as a match: the angle estimate of SimHash is
    theta = pi * ham / k, and a match needs cos(theta) > tau, i.e. ham < k * acos(tau) / pi."""
    if tau >= 1.0:
        return -1
    if tau <= -1.0:
        return k
    x = k * float(np.arccos(np.float64(tau))) / float(np.pi)
    h = int(np.ceil(x)) - 1          # largest integer strictly below x
    return max(-1, min(k, h))


def probe_simhash(bank: Bank, q_bf16, rq, tau: Optional[float] = None, h_out: Optional[np.ndarray] = None):
    """Probe by SimHash codes: nearest occupied key in Hamming distance (ties: lowest slot), hit iff the
    distance is within hamming_threshold(tau, k); reported score = cos(pi * ham / k) (float32).
    Everything after the decision is as in probe_fp.  Returns (ProbeResult, ham int32 [B])."""
    bank.tick += 1
    tau = bank.tau if tau is None else tau
    k = bank.fp_dim
    qb = simhash_bits(q_bf16)
    kb = simhash_bits(bank.fp)
    B = qb.shape[0]
    ham = np.full((B,), -1, dtype=np.int32)
    best = np.full((B,), -np.inf, dtype=np.float32)
    bslot = np.full((B,), -1, dtype=np.int32)
    occ = np.nonzero(bank.valid)[0]
    for b in range(B):
        if rq[b] <= 0:
            best[b] = 0.0
            continue
        if len(occ) == 0:
            continue
        d = (kb[occ] != qb[b][None, :]).sum(axis=1)
        i = int(np.argmin(d))                      # first minimum = lowest slot
        ham[b] = int(d[i])
        bslot[b] = int(occ[i])
        best[b] = np.float32(np.cos(np.pi * float(d[i]) / k))
    hmax = hamming_threshold(tau, k)
    hit = ((ham >= 0) & (ham <= hmax)).astype(np.uint8)
    slot = np.where(hit != 0, bslot, -1).astype(np.int32)
    hit_idx, miss_idx = compact(hit)
    if h_out is not None and bank.act is not None:
        for b in hit_idx.tolist():
            h_out[b] = bank.act[int(slot[b]) % bank.act_rows]
    touch(bank, slot[hit_idx])
    pr = ProbeResult(fp=q_bf16, rq=rq, score=best, second=None, best_slot=bslot, hit=hit, slot=slot,
                     hit_idx=hit_idx, miss_idx=miss_idx, tick=bank.tick)
    return pr, ham
