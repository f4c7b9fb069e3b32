"""The allocation-free fingerprint entry point against the ordinary one and against the oracle.

Some users of this library cannot let it allocate device memory: their host
application has already given the whole GPU to its own memory pool, or they
sit in a loop where the device-wide stall of cudaMalloc is unaffordable.  For
them llmcache_fingerprint_static keeps its scratch in a fixed array inside the
library.  This file checks, through the C ABI, that it returns what
llmcache_fingerprint returns (bit for bit: both launch the same two kernels in
the same shapes) and what the CPU oracle computes (within the fingerprint
tolerance) -- on two calls in a row, because the second call finds the array
as the first one left it --, that the second call leaves the amount of free
device memory unchanged, and that it refuses a batch that would not fit.  It is named to be collected last, so that a run stopping at the
first failure has already run every other test.
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


def _both(bank, h, dtype, dtype_code, n, d, k, proj, center, check_memory=False):
    B = h.shape[0]
    fp_a = torch.zeros((B, k), dtype=torch.bfloat16, device=DEV)
    rq_a = torch.zeros(B, dtype=torch.float32, device=DEV)
    fp_b = torch.full((B, k), 7.0, dtype=torch.bfloat16, device=DEV)
    rq_b = torch.full((B,), 7.0, dtype=torch.float32, device=DEV)
    L.llmcache_fingerprint(bank.handle, h, B, fp_a, rq_a)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    L.llmcache_fingerprint_static(h, dtype_code, B, n, d, k, proj, center, fp_b, rq_b)
    torch.cuda.synchronize()
    if check_memory:                       # the property the entry point exists for: it allocates nothing
        assert torch.cuda.mem_get_info()[0] == free_before
    assert L.llmcache_fingerprint_static_status() == L.OK
    # the two entry points launch the same kernels with the same launch shapes: identical bits
    assert torch.equal(fp_b.view(torch.int16), fp_a.view(torch.int16))
    assert torch.equal(rq_b.view(torch.int32), rq_a.view(torch.int32))
    # and against the oracle, with the tolerance the parity tests use for fingerprints (1e-3 relative over
    # the vector, one bf16 rounding step per element)
    host = h.cpu()
    fp_o, rq_o = O.fingerprint(U.bits(host) if dtype == "bf16" else host.numpy(), dtype,
                               None if proj is None else U.bits(proj), None if center is None else center.cpu().numpy())
    flipped = U.compare_fingerprints(U.bits(fp_b), rq_b.cpu().numpy(), fp_o, rq_o)
    assert flipped < 0.01


@pytest.mark.parametrize("dtype,n,d,k,use_proj", [("bf16", 384, 768, 256, True), ("f32", 128, 768, 768, False)])
def test_static_fingerprint_matches_the_bank_one_twice_in_a_row(dtype, n, d, k, use_proj):
    code = L.BF16 if dtype == "bf16" else L.F32
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    proj = synth.projection(d, k, 11, DEV) if use_proj else None
    center = synth.randn((d,), 12, DEV, scale=0.01) if use_proj else None
    bank = L.Bank(capacity=8, seq_len=n, d_model=d, fp_dim=k, max_batch=64, hidden_dtype=code, proj=proj, center=center)
    # first call: a full batch; second call right after it: a smaller, different batch with a zero row,
    # so anything stale left in the shared array by the first call would show
    h1 = synth.randn((64, n, d), 21, DEV, tdt)
    h2 = synth.randn((37, n, d), 22, DEV, tdt)
    h2[5] = 0
    _both(bank, h1, dtype, code, n, d, k, proj, center)
    _both(bank, h2, dtype, code, n, d, k, proj, center, check_memory=True)
    bank.close()


def test_static_fingerprint_refuses_what_does_not_fit_and_bad_arguments():
    n, d = 8, 4096
    B = L.FINGERPRINT_STATIC_MAX_FLOATS // d + 1            # one sequence too many even with a single split
    h = torch.zeros((B, n, d), dtype=torch.bfloat16, device=DEV)
    fp = torch.zeros((B, 64), dtype=torch.bfloat16, device=DEV)
    rq = torch.zeros(B, dtype=torch.float32, device=DEV)
    proj = synth.projection(d, 64, 1, DEV)
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_fingerprint_static(h, L.BF16, B, n, d, 64, proj, None, fp, rq)
    assert e.value.status == L.ERR_SHAPE and "limit" in str(e.value)
    L.llmcache_fingerprint_static(h[:16], L.BF16, 16, n, d, 64, proj, None, fp, rq)      # this much fits
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_fingerprint_static(h, L.BF16, 4, n, d, 100, proj, None, fp, rq)        # fp_dim not a multiple of 64
    assert e.value.status == L.ERR_SHAPE
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_fingerprint_static(None, L.BF16, 4, n, d, 64, proj, None, fp, rq)
    assert e.value.status == L.ERR_ARG
    torch.cuda.synchronize()
