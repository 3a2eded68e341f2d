"""GPU parity of the vocabulary-sharded entry points (fopd_shard_stats, fopd_shard_merge,
fopd_shard_loss_fwd_bwd): the merged result of any split of the vocabulary against the
fp64 CPU oracle's whole-row result, the partial sums themselves against the oracle's
plain definition, and the whole-row library path."""
import numpy as np
import pytest
import torch

from oracle import fopd_oracle as orc
from paper_2605_17862_b200 import binding as fb
from paper_2605_17862_b200 import synth

import _parity as par

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _chunks(wl, row_stride=None):
    return [synth.gen_chunk(wl, j, DEV, row_stride=row_stride) for j in range(wl.n_chunks)]


@pytest.mark.parametrize("name,parts", [("reasoning", 2), ("tool_use", 4), ("coding_agent", 3)])
def test_sharded_scaled_workloads(name, parts):
    wl = synth.WORKLOADS[name](scale=1 / 16)  # V = 9,496
    V = wl.V
    cuts = [0] + [8 * ((V * k // parts) // 8) for k in range(1, parts)] + [V]  # 16-byte aligned bf16 columns
    out = par.compare(_chunks(wl), wl.B, wl.tau, wl.H, grad_rows_per_chunk=64,
                      runner=par.gpu_run_vocab_sharded(cuts))
    print(name, cuts, out)


@pytest.mark.parametrize("dtype,cuts", [
    (torch.float32, [0, 4, 1000]),                 # a one-vector shard
    (torch.float32, [0, 500, 504, 996, 1000]),
    (torch.bfloat16, [0, 8, 16, 1000]),
    (torch.bfloat16, [0, 496, 1000]),
    (torch.bfloat16, [0, 1000]),                   # one holder: the sharded calls on whole rows
])
def test_sharded_uneven_splits_and_tails(dtype, cuts):
    rng = np.random.RandomState(len(cuts))
    B, V = 3, 1000
    lengths = np.array([10, 15, 12])
    n = int(lengths.sum())
    sid = np.repeat(np.arange(B, dtype=np.int32), lengths)
    mask = (rng.rand(n) > 0.2).astype(np.uint8)
    wl = synth.Workload("odd", B, V, dtype, n, sid, mask, np.array([0, 1, 2], np.int32), lengths.astype(np.int32),
                        sigma_s=2.0, seed=17)
    ch = synth.gen_chunk(wl, 0, DEV, row_stride=1008)
    # every shard must own some stored tokens, the first and last column included
    ch["tokens"][:4] = torch.tensor([0, V - 1, cuts[1] - 1, cuts[1] % V], dtype=torch.int32, device=DEV)
    par.compare([ch], B, wl.tau, wl.H, vocab=V, runner=par.gpu_run_vocab_sharded(cuts))


def test_sharded_chunks_with_an_empty_one():
    wl = synth.tiny(scale=1 / 8)
    ch = synth.gen_chunk(wl, 0, DEV)
    n = ch["tokens"].numel()
    chunks = [{k: v[a:b] for k, v in ch.items()} for a, b in ((0, 7), (7, 7), (7, n))]
    par.compare(chunks, wl.B, wl.tau, wl.H, runner=par.gpu_run_vocab_sharded([0, 8 * (wl.V // 24), wl.V]))


def test_partial_sums_match_the_oracle_definition():
    wl = synth.tiny(scale=1 / 8)
    ch = synth.gen_chunk(wl, 0, DEV)
    ch["mask"][3] = 0
    V, n = wl.V, ch["tokens"].numel()
    a, b = 1000, 3000
    part = torch.full((n, 8), float("nan"), device=DEV)
    fb.fopd_shard_stats(fb.Chunk(ch["student"][:, a:b], ch["teacher"][:, a:b], ch["behav_logprob"], ch["tokens"],
                                 ch["mask"], ch["sample_id"]), a, V, part)
    ref = orc.shard_partials(ch["student"][:, a:b].cpu().contiguous(), ch["teacher"][:, a:b].cpu().contiguous(),
                             ch["tokens"].cpu(), ch["mask"].cpu(), a)
    g = part.cpu().numpy().astype(np.float64)
    assert np.all(g[3] == 0.0)
    # the token's logits, the flag and the maxima are exact; the sums carry fp32 rounding
    assert np.array_equal(g[:, [0, 3, 5, 6, 7]], ref[:, [0, 3, 5, 6, 7]])
    assert np.allclose(g[:, [1, 4]], ref[:, [1, 4]], rtol=1e-5, atol=0)
    assert np.allclose(g[:, 2], ref[:, 2], rtol=1e-4, atol=1e-4)
    assert 0 < g[:, 7].sum() < n  # some tokens inside the shard, some outside


def test_sharded_and_whole_row_paths_agree():
    wl = synth.tool_use(scale=1 / 32)
    chunks = _chunks(wl)
    V = wl.V
    a = par.gpu_run(chunks, wl.B, wl.tau, wl.H)
    b = par.gpu_run_vocab_sharded([0, 8 * (V // 24), 8 * (V // 12), V])(chunks, wl.B, wl.tau, wl.H)
    assert a[3] == b[3] == 0
    assert torch.equal(a[0].acc[:, 0], b[0].acc[:, 0])
    assert torch.allclose(a[0].f, b[0].f, rtol=1e-5) and torch.allclose(a[0].loss, b[0].loss, rtol=1e-5)
    for x, y in zip(a[2], b[2]):
        assert torch.allclose(x.float(), y.float(), rtol=2e-2, atol=1e-7)


def test_token_in_no_part_and_bad_ids_are_reported():
    wl = synth.tiny(scale=1 / 8)
    ch = synth.gen_chunk(wl, 0, DEV)
    ch["tokens"][3] = wl.V  # outside the vocabulary: in no part
    ch["sample_id"][-1] = wl.B
    V = wl.V
    run = par.gpu_run_vocab_sharded([0, 8 * (V // 16), V])
    par.compare([ch], wl.B, wl.tau, wl.H, expect_bits=1 | 2, runner=run)
    # parts that do not cover the vocabulary: tokens in the gap are reported, the rest is unaffected
    n = ch["tokens"].numel()
    ch = synth.gen_chunk(wl, 0, DEV)
    ch["tokens"][5] = 2100
    part = torch.empty((2, n, 8), device=DEV)
    mk = lambda lo, hi: fb.Chunk(ch["student"][:, lo:hi], ch["teacher"][:, lo:hi], ch["behav_logprob"],
                                 ch["tokens"], ch["mask"], ch["sample_id"])
    fb.fopd_shard_stats(mk(0, 2000), 0, V, part[0])
    fb.fopd_shard_stats(mk(2200, V), 2200, V, part[1])
    acc = torch.zeros((wl.B, 4), dtype=torch.float64, device=DEV)
    ws = torch.empty((n, 4), device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    fb.fopd_shard_merge(part, ch["behav_logprob"], ch["tokens"], ch["mask"], ch["sample_id"], V, wl.B, acc, ws,
                        status=status)
    assert fb.fopd_check_status(status) & 1
    assert float(ws[5].abs().max()) == 0.0


def test_shard_argument_checks():
    wl = synth.tiny(scale=1 / 8)
    ch = synth.gen_chunk(wl, 0, DEV)
    n, V = ch["tokens"].numel(), wl.V
    part = torch.empty((n, 8), device=DEV)
    sh = fb.Chunk(ch["student"][:, 8:808], ch["teacher"][:, 8:808], ch["behav_logprob"], ch["tokens"], ch["mask"],
                  ch["sample_id"])
    with pytest.raises(fb.FopdError):  # shard reaches past the vocabulary
        fb.fopd_shard_stats(sh, V - 100, V, part)
    with pytest.raises(fb.FopdError):  # negative offset
        fb.fopd_shard_stats(sh, -8, V, part)
    bad = fb.Chunk(ch["student"][:, 3:803], ch["teacher"][:, 3:803], ch["behav_logprob"], ch["tokens"], ch["mask"],
                   ch["sample_id"])
    with pytest.raises(fb.FopdError):  # first column not 16-byte aligned
        fb.fopd_shard_stats(bad, 3, V, part)
    ws = torch.zeros((n, 4), device=DEV)
    coef = torch.ones(wl.B, device=DEV)
    with pytest.raises(fb.FopdError):  # gradient over the logits
        fb.fopd_shard_loss_fwd_bwd(sh, 8, V, wl.B, coef, ws, fb.params(**par.PARAMS), ch["student"][:, 8:808])
