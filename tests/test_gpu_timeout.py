"""The failure path of the kernels that wait on shared-memory rings, taken without a fault.

Every device-side wait is bounded.  With the producer thread of a kernel kept idle (a diagnostic knob) and the
bound lowered to a millisecond, the first wait of the kernel's consumers runs out: the kernel must record the
time-out in the object's status word, let anything in flight land, release its tensor memory and return, the
CUDA context must stay usable, and a fresh object on the same device must work as usual.  Nothing here traps,
asserts or touches a bad address: a wait simply ends early.
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
SHORT_NS = 1_000_000          # 1 ms


def small_bank(**kw):
    N, n, d, k, B = 256, 8, 128, 64, 8
    proj = synth.projection(d, k, 3, DEV)
    gb = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, hidden_dtype=L.BF16, proj=proj, tau=0.9, **kw)
    return gb, proj, (N, n, d, k, B)


def healthy_round_trip():
    """A fresh bank on the same device: insert, repeat, and compare with the oracle."""
    gb, proj, (N, n, d, k, B) = small_bank()
    ob = U.oracle_bank_like(gb, proj, None)
    bufs = L.ProbeBuffers(B, k, DEV)
    h = synth.randn((B, n, d), 41, DEV, torch.bfloat16)
    U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 42, DEV))
    r = U.lockstep_step(gb, ob, bufs, h, "bf16", synth.activations(B, n, d, 43, DEV))
    assert r["H"] == B and gb.status() == L.OK
    gb.close()


@pytest.mark.parametrize("call", ["probe", "probe_fp", "fingerprint"])
def test_expired_wait_is_reported_and_the_device_stays_usable(call):
    gb, proj, (N, n, d, k, B) = small_bank()
    bufs = L.ProbeBuffers(B, k, DEV)
    h = synth.randn((B, n, d), 31, DEV, torch.bfloat16)
    h_out = torch.zeros((B, n * d), dtype=torch.bfloat16, device=DEV)
    # a healthy probe + commit first, so that the scan has keys to walk
    gb.probe(h, bufs, h_out=h_out)
    gb.commit(synth.activations(B, n, d, 32, DEV), bufs, h_out=h_out)
    assert gb.status() == L.OK
    gb.debug_knobs(SHORT_NS, L.KNOB_PRODUCER_IDLE)
    if call == "probe":              # pooling pass, projection and scan all starve
        gb.probe(h, bufs, h_out=h_out)
    elif call == "probe_fp":         # the scan alone
        gb.probe_fp(bufs, B, h_out=h_out)
    else:                            # pooling pass and projection
        L.llmcache_fingerprint(gb.handle, h, B, bufs.fp, bufs.rq)
    torch.cuda.synchronize()         # returns: nothing hangs
    assert gb.status() == L.ERR_TIMEOUT
    assert "wait" in L.strerror(L.ERR_TIMEOUT)
    gb.close()
    healthy_round_trip()


def test_expired_wait_in_the_row_movers_and_the_layer():
    n, d, k, B, N = 8, 128, 64, 8, 64
    proj = synth.projection(d, k, 3, DEV)
    gb = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=k, max_batch=B, hidden_dtype=L.BF16, proj=proj, fused_pool=1)
    bufs = L.ProbeBuffers(B, k, DEV)
    pooled = torch.zeros((B, d), dtype=torch.float32, device=DEV)
    h = synth.randn((B, n, d), 51, DEV, torch.bfloat16)
    h_out = torch.zeros((B, n * d), dtype=torch.bfloat16, device=DEV)
    gb.pool_out(pooled)
    gb.probe(h, bufs, h_out=h_out)
    gb.debug_knobs(SHORT_NS, L.KNOB_PRODUCER_IDLE)        # the moving pass of the commit starves
    gb.commit(synth.activations(B, n, d, 52, DEV), bufs, h_out=h_out)
    torch.cuda.synchronize()
    assert gb.status() == L.ERR_TIMEOUT
    gb.close()
    # the layer's dense kernels
    w = synth.layer_weights(128, 256, 61, DEV)
    layer = L.Layer(w, heads=2, seq_len=16, max_seqs=4)
    x = synth.randn((4, 16, 128), 62, DEV, torch.bfloat16)
    out = torch.zeros_like(x)
    layer.forward(x, out)
    assert layer.status() == L.OK
    layer.debug_knobs(SHORT_NS, L.KNOB_PRODUCER_IDLE)
    layer.forward(x, out)
    torch.cuda.synchronize()
    assert layer.status() == L.ERR_TIMEOUT
    layer.debug_knobs(0, 0)                                # knobs off: the kernels run again (the status stays set)
    out2 = torch.zeros_like(x)
    layer.forward(x, out2)
    torch.cuda.synchronize()
    assert torch.isfinite(out2.float()).all()
    layer.close()
    healthy_round_trip()
