"""Fingerprint (Sec. IV-B) on widths that do not line up with the kernels' tiles.

The projection runs on 16-row tensor-core steps, 64-column TMA boxes and 8-column tiles dealt to 16 warps;
the shapes here leave ragged ends in each of them (d_model not a multiple of 16, fp_dim of 64 .. 1088
columns, batches that do not fill a group of 8 sequences, one sequence, more rows of the projection matrix
than one refill of the operand holds), with and without a centring vector, from hidden states and from
given position means.  Compared element by element with the oracle under the fingerprint tolerance.
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


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("B,n,d,k,use_center", [
    (1, 3, 72, 64, False),        # one sequence, 4.5 tensor-core steps of rows
    (9, 7, 136, 192, True),       # 24 column tiles over 16 warps
    (65, 5, 200, 320, True),      # 40 column tiles, 4 per warp, six warps idle
    (13, 4, 1000, 1088, False),   # 17 boxes of 64 columns, 8 tiles per warp
    (21, 2, 2344, 128, True),     # more rows than one refill of the operand (and not a multiple of 16)
])
def test_projected_fingerprint_ragged_shapes(B, n, d, k, use_center, dtype):
    if dtype == "f32" and d > 3840:
        pytest.skip("f32 hidden states stop at d_model 3840")
    code = L.BF16 if dtype == "bf16" else L.F32
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    proj = synth.projection(d, k, 100 + d, DEV)
    center = synth.randn((d,), 200 + d, DEV, scale=0.05) if use_center else None
    bank = L.Bank(capacity=4, seq_len=n, d_model=d, fp_dim=k, max_batch=B, hidden_dtype=code, proj=proj, center=center)
    h = synth.randn((B, n, d), 300 + d, DEV, tdt)
    if B > 2:
        h[2] = 0                                             # a degenerate sequence in the middle of a group
    fp = torch.full((B, k), 3.0, dtype=torch.bfloat16, device=DEV)
    rq = torch.full((B,), 3.0, dtype=torch.float32, device=DEV)
    L.llmcache_fingerprint(bank.handle, h, B, fp, rq)
    torch.cuda.synchronize()
    assert bank.status() == L.OK
    hb = U.bits(h) if dtype == "bf16" else h.cpu().numpy()
    c = center.cpu().numpy() if use_center else None
    want_fp, want_rq = O.fingerprint(hb, dtype, U.bits(proj), c)
    if use_center:
        # a zero sequence minus the centring vector is not degenerate; without it the fingerprint is zero
        assert want_rq[2] > 0 if B > 2 else True
    elif B > 2:
        assert want_rq[2] == 0 and float(rq[2]) == 0.0
    U.compare_fingerprints(U.bits(fp), rq.cpu().numpy(), want_fp, want_rq)

    # the same from given position means (strided source: the second half of a [B, 2d] array)
    means = torch.zeros((B, 2 * d), dtype=torch.float32, device=DEV)
    bank.pool(h, means[:, d:])
    fp2 = torch.zeros((B, k), dtype=torch.bfloat16, device=DEV)
    rq2 = torch.zeros(B, dtype=torch.float32, device=DEV)
    L.llmcache_fingerprint_pooled(bank.handle, means[:, d:], 2 * d, B, fp2, rq2)
    torch.cuda.synchronize()
    assert bank.status() == L.OK
    U.compare_fingerprints(U.bits(fp2), rq2.cpu().numpy(), want_fp, want_rq)
    bank.close()


def test_input_stable_promise_changes_nothing_but_the_start_of_the_pooling_pass():
    """With llmcache_bank_input_stable the pooling pass streams its input before the preceding kernel of the
    stream has finished; the fingerprints, decisions and bank state must be bit-identical to the ordinary path."""
    N, n, d, k, B = 256, 96, 256, 128, 70
    proj = synth.projection(d, k, 5, DEV)
    mk = lambda: L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, hidden_dtype=L.BF16, proj=proj, tau=0.9)
    ga, gb = mk(), mk()
    gb.input_stable(True)
    ba, bb = L.ProbeBuffers(B, k, DEV), L.ProbeBuffers(B, k, DEV)
    big = torch.empty(64 * 1024 * 1024, dtype=torch.uint8, device=DEV)
    for step in range(3):
        h = synth.randn((B, n, d), 40 + step % 2, DEV, torch.bfloat16)       # the third batch repeats the first
        mo = synth.activations(B, n, d, 50 + step, DEV)
        for g, b in ((ga, ba), (gb, bb)):
            big.fill_(step)                                                   # a kernel that is still running when the probe is enqueued
            g.probe(h, b)
            g.commit(mo, b)
        torch.cuda.synchronize()
        assert torch.equal(ba.fp.view(torch.int16), bb.fp.view(torch.int16))
        assert torch.equal(ba.rq.view(torch.int32), bb.rq.view(torch.int32))
        assert torch.equal(ba.hit, bb.hit) and torch.equal(ba.slot, bb.slot)
    for what in (L.WHAT_FP, L.WHAT_VALID, L.WHAT_LAST_USE, L.WHAT_RATE):
        assert torch.equal(ga.export(what), gb.export(what))
    assert int(ba.counts[0]) == B and ga.status() == L.OK and gb.status() == L.OK
    ga.close()
    gb.close()
