"""Probes of a handful of sequences with a projection matrix (the paper measures at batch 1), in lock step with
the oracle:
empty bank, repeats that hit, several sequences of a batch matching the same entry, a degenerate (all-zero)
sequence, centring, the >= comparison, fp32 inputs, widths that leave ragged ends, a bank of one slot."""
import numpy as np
import pytest
import torch

from oracle import llmcache_oracle as O
from paper_2512_16843_b200 import binding as L
from paper_2512_16843_b200 import synth
from tests import parity_util as U
from tests.test_gpu_parity import make_pair, rand_h

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("N,n,d,k,B,dtype,use_center,cmp,policy", [
    (64, 16, 128, 64, 1, "bf16", False, L.GT, L.LRU),
    (2048, 128, 768, 256, 1, "bf16", False, L.GT, L.LRU_STALENESS),      # the paper's batch 1 x seq_len 128
    (300, 37, 192, 128, 3, "f32", True, L.GT, L.LRU_STALENESS),
    (1000, 5, 768, 256, 8, "bf16", True, L.GE, L.LRU),
    (7, 3, 136, 192, 5, "bf16", False, L.GT, L.LRU_STALENESS),
    (1, 4, 64, 64, 2, "f32", False, L.GT, L.LRU),
    (513, 9, 1000, 320, 6, "bf16", False, L.GT, L.LRU_STALENESS),
])
def test_small_batch_probe_lockstep(N, n, d, k, B, dtype, use_center, cmp, policy):
    proj = synth.projection(d, k, 400 + d, DEV)
    center = synth.randn((d,), 401 + d, DEV, scale=0.05) if use_center else None
    gb, ob = make_pair(N, n, d, k, B, dtype, proj, center, cmp=cmp, policy=policy)
    bufs = L.ProbeBuffers(B, k, DEV)
    base = rand_h(B, n, d, 410, dtype)
    hits_seen = 0
    for step in range(5):
        h = rand_h(B, n, d, 420 + step, dtype)
        if step >= 1:
            h[0] = base[0]                                   # comes back every step
        if step >= 2 and B > 1:
            h[1] = base[0]                                   # two sequences of the batch match the same entry
        if step == 3 and B > 2:
            h[2] = 0                                         # degenerate unless a centring vector shifts it
        if step == 0:
            h = base.clone()
        r = U.lockstep_step(gb, ob, bufs, h, dtype, synth.activations(B, n, d, 430 + step, DEV))
        hits_seen += r["H"]
    if N >= B:
        assert hits_seen >= 4                                # the repeats did hit
    gb.close()


def test_small_batch_tau_and_threshold_equality():
    """tau given per call; with >= an exact repeat at tau = its own score hits, with > it does not."""
    N, n, d, k, B = 32, 8, 128, 64, 2
    proj = synth.projection(d, k, 55, DEV)
    for cmp in (L.GT, L.GE):
        gb, ob = make_pair(N, n, d, k, B, "bf16", proj, None, cmp=cmp)
        bufs = L.ProbeBuffers(B, k, DEV)
        h = rand_h(B, n, d, 56, "bf16")
        U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 57, DEV))
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 58, DEV), do_commit=False)
        assert r["H"] == B
        s = float(bufs.score[0])
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 59, DEV), tau=s, do_commit=False)
        assert bool(bufs.hit[0]) == (cmp == L.GE)
        r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 60, DEV), tau=1.5, do_commit=False)
        assert r["H"] == 0
        gb.close()
