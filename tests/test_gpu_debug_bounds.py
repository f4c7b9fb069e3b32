"""The range-checking build of the library (-DLLMCACHE_DEBUG_BOUNDS).

That build checks every slot, row and batch index that the row movers, the decision and the victim selection
compute before it is used; a violation is recorded in the bank's status word and the access is skipped.  The
whole GPU suite is meant to be run once against it (LLMCACHE_LIB=.../libllmcache_dbg.so python -m pytest tests
-m gpu): every test's status checks then also assert that no index ever left its range.  The test below runs
only against that build: it hands the commit an index list with one entry out of range and expects
LLMCACHE_ERR_BOUNDS, not a fault (the ordinary build has no such check, so there the test is skipped).
"""
import pytest
import torch

from paper_2512_16843_b200 import binding as L
from paper_2512_16843_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_out_of_range_index_is_reported_and_skipped():
    if not L.llmcache_debug_bounds_build():
        pytest.skip("needs the library built with -DLLMCACHE_DEBUG_BOUNDS")
    N, n, d, B = 64, 4, 64, 16
    gb = L.Bank(capacity=N, seq_len=n, d_model=d, fp_dim=d, max_batch=B)
    bufs = L.ProbeBuffers(B, d, DEV)
    h = synth.randn((B, n, d), 5, DEV, torch.bfloat16)
    h_out = torch.zeros((B, n * d), dtype=torch.bfloat16, device=DEV)
    gb.probe(h, bufs, h_out=h_out)
    torch.cuda.synchronize()
    assert gb.status() == L.OK and int(bufs.counts[1]) == B
    bufs.miss_idx[3] = B + 1000                      # what a broken compaction would produce
    before = h_out.clone()
    gb.commit(synth.activations(B, n, d, 6, DEV), bufs, h_out=h_out)
    torch.cuda.synchronize()
    assert gb.status() == L.ERR_BOUNDS
    assert "range" in L.strerror(L.ERR_BOUNDS)
    assert torch.equal(h_out[3], before[3])          # the row of the bad entry was not written anywhere valid
    gb.close()
