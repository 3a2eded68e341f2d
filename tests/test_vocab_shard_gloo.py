"""World-size-2 gloo test of the one exchange of the vocabulary-sharded path: each
rank holds half of the columns, forms its partial sums (with the CPU oracle here:
the CUDA kernels need a GPU), pipeline.gather_parts brings all parts to every rank
in rank order, and the merged result equals the whole-row statistics on both ranks."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from oracle import fopd_oracle as orc
    from paper_2605_17862_b200 import pipeline as pl
    from paper_2605_17862_b200 import synth

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.tiny(scale=1 / 16)          # the same seeded rows on both ranks
    ch = synth.gen_chunk(wl, 0)
    V = wl.V
    cuts = [0, 8 * (V // 24), V]           # uneven halves
    a, b = cuts[rank], cuts[rank + 1]
    mine = orc.shard_partials(ch["student"][:, a:b].contiguous(), ch["teacher"][:, a:b].contiguous(), ch["tokens"],
                              ch["mask"], a)
    parts = pl.gather_parts(torch.as_tensor(mine))
    assert parts.shape == (world, ch["tokens"].numel(), 8)
    assert torch.equal(parts[rank], torch.as_tensor(mine))
    lse_s, lse_t, kl, sy, ty, found = orc.merge_partials(parts.numpy())
    whole = orc.token_stats(ch["student"], ch["teacher"], ch["tokens"], ch["behav_logprob"], ch["mask"],
                            ch["sample_id"], wl.B)
    ok = whole.valid.astype(bool)
    err = max(np.abs(lse_s - whole.lse_s)[ok].max(), np.abs(kl - whole.kl)[ok].max(),
              np.abs((sy - lse_s) - whole.lp_s)[ok].max(), np.abs((ty - lse_t) - whole.lp_t)[ok].max())
    out[rank] = (float(err), float(found[ok].min()), float(found[ok].max()), float(parts.double().sum()))
    dist.destroy_process_group()


def test_partial_sums_reach_every_rank_in_rank_order():
    world, port = 2, 30500 + os.getpid() % 1000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        err, fmin, fmax, _ = res[rank]
        assert err < 1e-11 and fmin == fmax == 1.0
    assert res[0][3] == res[1][3]  # both ranks hold the same stack of parts


def test_single_process_gather_is_a_copy():
    sys.path.insert(0, ROOT)
    from paper_2605_17862_b200 import pipeline as pl

    x = torch.arange(24, dtype=torch.float32).reshape(3, 8)
    assert torch.equal(pl.gather_parts(x), x[None])
