"""Seeded random cases through every path of the library (cached statistics, on-chip kernel,
vocabulary shards, host buffers with the large and the small workspace), each compared with
the fp64 CPU oracle element by element: random vocabulary sizes (one column to several
clusters' worth, with and without a ragged tail), row pitches, dtypes, sample lengths
(empty samples included), masks, chunk splits (empty chunks included), gate thresholds,
supervision drifts, and now and then a token or sample id out of range."""
import numpy as np
import pytest
import torch

from paper_2605_17862_b200 import synth

import _parity as par
import test_gpu_host_step as host_step

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MODES = ("cached", "on_chip", "sharded", "host_resident", "host_small_workspace")
VOCABS = (1, 3, 17, 100, 1000, 4099, 9496, 20000, 32000, 40961, 65544, 70001)


def _case(seed):
    rng = np.random.RandomState(seed)
    dtype = (torch.bfloat16, torch.float32)[rng.randint(2)]
    per = 8 if dtype == torch.bfloat16 else 4  # columns per 16 bytes
    V = int(VOCABS[rng.randint(len(VOCABS))])
    stride = ((V + per - 1) // per + int(rng.choice([0, 0, 1, 3]))) * per
    B = int(rng.randint(1, 7))
    lengths = rng.randint(0, 40, B)
    if lengths.sum() == 0:
        lengths[0] = 5
    n = int(lengths.sum())
    sid = np.repeat(np.arange(B, dtype=np.int32), lengths)
    mask = (rng.rand(n) > rng.choice([0.0, 0.3, 0.7])).astype(np.uint8)
    wl = synth.Workload("random", B, V, dtype, n, sid, mask, rng.randint(0, 5, B).astype(np.int32),
                        np.maximum(lengths, 1).astype(np.int32), sigma_s=float(rng.choice([1.0, 3.0])),
                        sigma_t=float(rng.choice([0.5, 2.0])), seed=seed)
    whole = synth.gen_chunk(wl, 0, DEV, row_stride=stride)
    bits = 0  # device status word the case must end with
    if rng.rand() < 0.25:  # a stored token outside the vocabulary (reported only on an aligned row)
        r = int(rng.randint(0, n))
        whole["tokens"][r] = int(rng.choice([-1, V, V + 5]))
        if int(whole["mask"][r]) != 0:
            bits |= 1
    if rng.rand() < 0.15:  # a sample id outside the batch, on the last row so that ids stay sorted
        whole["sample_id"][n - 1] = B
        bits |= 2
    cuts = sorted(set([0, n] + list(rng.randint(0, n + 1, rng.randint(0, 3)))))
    if rng.rand() < 0.2:
        cuts = sorted(cuts + [cuts[len(cuts) // 2]])  # an empty chunk
    chunks = [{k: v[a:b] for k, v in whole.items()} for a, b in zip(cuts[:-1], cuts[1:])]
    params = dict(par.PARAMS, xi=float(rng.choice([0.0, 0.05, 0.15])))
    d_sup = None if rng.rand() < 0.5 else (rng.rand(B) * 0.3).astype(np.float32)
    shard_cuts = [0, V]
    if V >= 2 * per:
        inner = {per * int(x) for x in rng.randint(1, max(2, V // per), rng.randint(1, 4))}
        shard_cuts = [0] + sorted(c for c in inner if c < V) + [V]
    return wl, V, chunks, params, d_sup, shard_cuts, bits, MODES[rng.randint(len(MODES))]


@pytest.mark.parametrize("seed", range(2000, 2100))
def test_random_case(seed):
    wl, V, chunks, params, d_sup, shard_cuts, bits, mode = _case(seed)
    if mode in ("cached", "on_chip"):
        par.compare(chunks, wl.B, wl.tau, wl.H, d_sup=d_sup, params=params, use_row_ws=(mode == "cached"), vocab=V,
                    expect_bits=bits)
    elif mode == "sharded":
        par.compare(chunks, wl.B, wl.tau, wl.H, d_sup=d_sup, params=params, vocab=V,
                    runner=par.gpu_run_vocab_sharded(shard_cuts), expect_bits=bits)
    else:
        host = [{k: v.cpu().pin_memory() for k, v in c.items()} for c in chunks]
        host_step._check(host, wl.B, wl.tau, wl.H, d_sup=d_sup, params=params, resident=(mode == "host_resident"),
                         vocab=V, expect_bits=bits)
