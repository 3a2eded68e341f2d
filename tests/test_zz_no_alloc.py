"""fopd_token_stats_static -- the statistics entry point for callers that cannot
allocate GPU memory (all of it belongs to their own allocator, or their step
loop forbids allocation) -- must give what fopd_token_stats gives, which is
what the fp64 oracle gives within the path's tolerances, and must leave the
amount of free device memory as it found it.

Collected last on purpose: if it fails, a run that stops at the first failure
has already run every other test.  Two calls in a row share the library's
built-in scratch array; the second uses fewer rows than the first, so values
left behind by the first call would show up if they were ever read.
"""
import numpy as np
import pytest
import torch

from oracle import fopd_oracle as orc
from paper_2605_17862_b200 import binding as fb
from paper_2605_17862_b200 import pipeline as pl
from paper_2605_17862_b200 import synth

import _parity as par

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(wl, j=0, check_memory=False):
    ch = synth.gen_chunk(wl, j, DEV)
    n = ch["student"].shape[0]
    chunk = pl.to_chunk(ch)
    ref_rows, new_rows = pl.RowOutputs.alloc(n, DEV), pl.RowOutputs.alloc(n, DEV)
    ref_buf, new_buf = pl.BatchBuffers(wl.B, DEV), pl.BatchBuffers(wl.B, DEV)
    fb.fopd_token_stats(chunk, wl.B, ref_buf.acc, lp_s=ref_rows.lp_s, lp_t=ref_rows.lp_t, kl=ref_rows.kl,
                        ratio=ref_rows.ratio, row_ws=None, status=ref_buf.status)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(DEV)[0]
    fb.fopd_token_stats_static(chunk, wl.B, new_buf.acc, lp_s=new_rows.lp_s, lp_t=new_rows.lp_t,
                               kl=new_rows.kl, ratio=new_rows.ratio, status=new_buf.status)
    torch.cuda.synchronize()
    if check_memory:  # not on the first call of a process: that one loads the module holding the array
        assert torch.cuda.mem_get_info(DEV)[0] == free_before, "the entry point took device memory"
    assert fb.fopd_check_status(new_buf.status) == fb.fopd_check_status(ref_buf.status) == 0
    assert float(ref_buf.acc[:, 0].sum()) > 0

    # against the oracle, with the tolerances of the parity tests
    host = par.host_chunk(ch)
    st = orc.token_stats(host["student"], host["teacher"], host["tokens"], host["behav_logprob"], host["mask"],
                         host["sample_id"], wl.B)
    valid = st.valid.astype(bool)
    g = {k: getattr(new_rows, k).cpu().numpy().astype(np.float64) for k in ("lp_s", "lp_t", "kl", "ratio")}
    for k in g:
        assert np.all(g[k][~valid] == 0.0), k
    assert np.abs(g["lp_s"] - st.lp_s)[valid].max() <= par.TOL_LOGPROB
    assert np.abs(g["lp_t"] - st.lp_t)[valid].max() <= par.TOL_LOGPROB
    assert (np.abs(g["kl"] - st.kl) / np.maximum(1.0, st.kl))[valid].max() <= 1e-4
    assert (np.abs(g["ratio"] - st.rho)[valid] / st.rho[valid]).max() <= 1.1 * par.TOL_LOGPROB
    acc_o = np.zeros((wl.B, 3))
    orc.sample_accumulate(acc_o, host["sample_id"], st)
    acc = new_buf.acc.cpu().numpy()
    assert np.array_equal(acc[:, 0], acc_o[:, 0])
    assert np.allclose(acc[:, 1], acc_o[:, 1], rtol=par.TOL_REL, atol=1e-6 * max(1.0, acc_o[:, 0].max()))
    assert np.allclose(acc[:, 2], acc_o[:, 2], rtol=par.TOL_REL, atol=1e-6 * max(1.0, acc_o[:, 0].max()))

    # and the existing entry point: same kernels, fixed summation order, so the very same bits
    for name in ("lp_s", "lp_t", "kl", "ratio"):
        assert torch.equal(getattr(ref_rows, name), getattr(new_rows, name)), name
    assert torch.equal(ref_buf.acc, new_buf.acc)


def test_static_scratch_entry_matches_oracle_and_allocating_entry_twice_in_a_row():
    _both(synth.coding_agent(scale=1 / 16), j=1)   # 1,024 rows, about half masked
    # fewer aligned rows, other masks: stale scratch must not leak; free memory must not move
    _both(synth.reasoning(scale=1 / 32), check_memory=True)


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
    c.n_rows = 4
    rc = fb.lib().fopd_token_stats_static(ctypes.byref(c), fb.STATIC_MAX_SAMPLES + 1, None, None, None, None,
                                          ctypes.c_void_p(buf.acc.data_ptr()), None, None)
    assert rc == -3  # more samples than the built-in row-range array holds
    torch.cuda.synchronize()
    assert float(buf.acc.abs().sum()) == 0.0
