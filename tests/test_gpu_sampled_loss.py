"""GPU parity of the sampled-token form of the token loss (FOPD_LOSS_SAMPLED_KL: the
importance-weighted reverse KL on the stored token, Sec. 5 / Appendix B) against the
fp64 CPU oracle: the five workloads at sizes the oracle finishes in seconds, cached and
uncached row statistics, odd vocabularies, gates, bad ids, and the entry points that do
not take this form."""
import numpy as np
import pytest
import torch

from paper_2605_17862_b200 import binding as fb
from paper_2605_17862_b200 import pipeline as pl
from paper_2605_17862_b200 import synth

import _parity as par

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SAMPLED = fb.LOSS_SAMPLED_KL


def _chunks(wl, row_stride=None):
    return [synth.gen_chunk(wl, j, DEV, row_stride=row_stride) for j in range(wl.n_chunks)]


@pytest.mark.parametrize("use_row_ws", [True, False])
@pytest.mark.parametrize("name,scale", [("tiny", 1.0), ("reasoning", 1 / 16), ("tool_use", 1 / 16),
                                        ("coding_agent", 1 / 16)])
def test_workloads_scaled(name, scale, use_row_ws):
    wl = synth.WORKLOADS[name](scale=scale)
    out = par.compare(_chunks(wl), wl.B, wl.tau, wl.H, use_row_ws=use_row_ws, grad_rows_per_chunk=48,
                      loss_kind=SAMPLED)
    print(name, use_row_ws, out)


def test_roofline_point_scaled():
    wl = synth.roofline_point(512, 32000)
    print(par.compare(_chunks(wl), wl.B, wl.tau, wl.H, grad_rows_per_chunk=32, loss_kind=SAMPLED))


@pytest.mark.parametrize("V,stride,dtype", [(1, 8, torch.bfloat16), (7, 8, torch.bfloat16), (33, 36, torch.float32),
                                            (4099, 4104, torch.bfloat16), (70001, 70008, torch.bfloat16)])
def test_odd_vocabularies_and_pitches(V, stride, dtype):
    rng = np.random.RandomState(V)
    B, lengths = 3, np.array([9, 17, 14])
    n = int(lengths.sum())
    sid = np.repeat(np.arange(B, dtype=np.int32), lengths)
    mask = (rng.rand(n) > 0.25).astype(np.uint8)
    wl = synth.Workload("odd", B, V, dtype, n, sid, mask, np.array([0, 1, 2], np.int32), lengths.astype(np.int32),
                        seed=V % 977)
    ch = synth.gen_chunk(wl, 0, DEV, row_block=8, row_stride=stride)
    ch["student"][:, V:] = 1e4   # pitch padding must not be read
    ch["teacher"][:, V:] = -1e4
    for use_ws in (True, False):
        print(V, par.compare([ch], B, wl.tau, wl.H, use_row_ws=use_ws, vocab=V, loss_kind=SAMPLED))


def test_stationary_point_and_lag_only_weighting():
    """Teacher = student and behaviour = current: loss and gradient vanish; alpha = beta = 0 is the
    lag-only weighting of Appendix B with this form of the loss."""
    wl = synth.tool_use(scale=1 / 32)
    chunks = _chunks(wl)
    for c in chunks:
        c["teacher"] = c["student"].clone()
        lp = torch.log_softmax(c["student"].float(), 1).gather(1, c["tokens"].long().clamp(0).unsqueeze(1)).squeeze(1)
        c["behav_logprob"] = lp
    buf, rows, dl, bits = par.gpu_run(chunks, wl.B, wl.tau, wl.H, loss_kind=SAMPLED)
    assert bits == 0 and abs(float(buf.loss)) < 1e-6
    assert max(float(d.abs().max()) for d in dl) < 1e-8
    chunks = _chunks(wl)
    par.compare(chunks, wl.B, wl.tau, wl.H, params=dict(par.PARAMS, alpha=0.0, beta=0.0), grad_rows_per_chunk=16,
                loss_kind=SAMPLED)


def test_bad_ids_and_gated_samples():
    wl = synth.coding_agent(scale=1 / 32)   # staleness up to 8: gated samples
    chunks = _chunks(wl)
    tok = chunks[0]["tokens"].clone()
    aligned = torch.nonzero(chunks[0]["mask"]).flatten()   # a bad token only counts on an aligned row
    tok[aligned[2]] = wl.V
    tok[aligned[7]] = -3
    chunks[0]["tokens"] = tok
    out = par.compare(chunks, wl.B, wl.tau, wl.H, expect_bits=1, grad_rows_per_chunk=32, loss_kind=SAMPLED)
    buf, *_ = par.gpu_run(chunks, wl.B, wl.tau, wl.H, loss_kind=SAMPLED)
    assert int((buf.w == 0).sum()) >= 1
    print(out)


def test_entry_points_that_take_the_full_vocabulary_form_only():
    wl = synth.tiny(scale=1 / 8)
    ch = synth.gen_chunk(wl, 0, DEV)
    c = pl.to_chunk(ch, loss_kind=SAMPLED)
    part = torch.empty((ch["tokens"].numel(), 8), dtype=torch.float32, device=DEV)
    with pytest.raises(fb.FopdError) as e:
        fb.fopd_shard_stats(c, 0, wl.V, part)
    assert e.value.code == -9
    bad = pl.to_chunk(ch, loss_kind=5)
    buf = pl.BatchBuffers(wl.B, DEV)
    with pytest.raises(fb.FopdError) as e:
        fb.fopd_token_stats(bad, wl.B, buf.acc)
    assert e.value.code == -9
