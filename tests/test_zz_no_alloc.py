"""fopd_token_stats_static -- the statistics entry point for callers that cannot
allocate GPU memory (all of it belongs to their own allocator, or their step
loop forbids allocation) -- must give what fopd_token_stats gives.

Collected last on purpose: if it fails, a run that stops at the first failure
has already run every other test.  Two calls in a row share the library's
built-in scratch array; the second uses fewer rows than the first, so values
left behind by the first call would show up if they were ever read.
"""
import pytest
import torch

from paper_2605_17862_b200 import binding as fb
from paper_2605_17862_b200 import pipeline as pl
from paper_2605_17862_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(wl, j=0):
    ch = synth.gen_chunk(wl, j, DEV)
    n = ch["student"].shape[0]
    chunk = pl.to_chunk(ch)
    ref_rows, new_rows = pl.RowOutputs.alloc(n, DEV), pl.RowOutputs.alloc(n, DEV)
    ref_buf, new_buf = pl.BatchBuffers(wl.B, DEV), pl.BatchBuffers(wl.B, DEV)
    fb.fopd_token_stats(chunk, wl.B, ref_buf.acc, lp_s=ref_rows.lp_s, lp_t=ref_rows.lp_t, kl=ref_rows.kl,
                        ratio=ref_rows.ratio, row_ws=None, status=ref_buf.status)
    fb.fopd_token_stats_static(chunk, wl.B, new_buf.acc, lp_s=new_rows.lp_s, lp_t=new_rows.lp_t,
                               kl=new_rows.kl, ratio=new_rows.ratio, status=new_buf.status)
    torch.cuda.synchronize()
    assert fb.fopd_check_status(new_buf.status) == fb.fopd_check_status(ref_buf.status) == 0
    assert float(ref_buf.acc[:, 0].sum()) > 0
    # same kernels, fixed summation order: identical, which is inside every tolerance used elsewhere
    for name in ("lp_s", "lp_t", "kl", "ratio"):
        a, b = getattr(ref_rows, name), getattr(new_rows, name)
        assert torch.allclose(a, b, rtol=0, atol=1e-3) and torch.equal(a, b), name
    assert torch.allclose(ref_buf.acc, new_buf.acc, rtol=1e-4) and torch.equal(ref_buf.acc, new_buf.acc)


def test_static_scratch_entry_matches_allocating_entry_twice_in_a_row():
    _both(synth.coding_agent(scale=1 / 16), j=1)   # 1,024 rows, about half masked
    _both(synth.reasoning(scale=1 / 32))           # fewer aligned rows, other masks: stale scratch must not leak


def test_static_scratch_entry_rejects_oversized_chunks():
    wl = synth.tiny(scale=1 / 8)
    ch = pl.to_chunk(synth.gen_chunk(wl, 0, DEV))
    c = ch.c_struct()
    c.n_rows = fb.STATIC_MAX_ROWS + 1  # rejected on the host before anything is enqueued
    import ctypes
    buf = pl.BatchBuffers(wl.B, DEV)
    rc = fb.lib().fopd_token_stats_static(ctypes.byref(c), wl.B, None, None, None, None,
                                          ctypes.c_void_p(buf.acc.data_ptr()), None, None)
    assert rc == -3
    torch.cuda.synchronize()
    assert float(buf.acc.abs().sum()) == 0.0
