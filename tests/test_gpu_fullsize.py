"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The fp64 CPU oracle runs its whole measurement phase over every row (chunk by
chunk on host copies of the same bits; tens of seconds on the host cores), so
every per-row output, the per-sample sums, freshness, gate, weights and the loss
are compared against it with nothing taken from the CUDA path.  The gradient is
compared on a seeded sample of rows that the oracle computes one by one -- always
including the first and last row of every chunk and the rows on both sides of
every sample boundary -- and, for all rows, through properties that hold at any
size: rows that are not differentiated are exactly +0, every differentiated row
sums to zero.  Chunks are streamed (generated, used, freed) exactly as the
chunked configurations say.
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
ROWS_PER_CHUNK = 12  # random rows per chunk on top of the mandatory ones


def _sample_rows(sid, n, rng):
    edges = np.nonzero(np.diff(sid))[0]
    must = np.concatenate([[0, n - 1], edges, edges + 1])
    extra = rng.choice(n, size=min(n, ROWS_PER_CHUNK), replace=False)
    return np.unique(np.concatenate([must, extra])).astype(np.int64)


def _sub_chunk(ch, rows):
    idx = torch.as_tensor(rows, device=ch["student"].device)
    return {k: v[idx].cpu() for k, v in ch.items()}


_ORACLE_CACHE = {}


def _oracle_measurement(wl):
    """The oracle's measurement phase over EVERY row of the workload, chunk by chunk on host
    copies of the same generated bits (cached per workload: two tests share `reasoning`)."""
    if wl.name in _ORACLE_CACHE:
        return _ORACLE_CACHE[wl.name]
    rng = np.random.default_rng(wl.seed)
    acc = np.zeros((wl.B, 3))
    stats, picks, subs = [], [], []
    for j in range(wl.n_chunks):
        ch = synth.gen_chunk(wl, j, DEV)
        host = {k: v.cpu() for k, v in ch.items()}
        st = orc.token_stats(host["student"], host["teacher"], host["tokens"], host["behav_logprob"], host["mask"],
                             host["sample_id"], wl.B)
        orc.sample_accumulate(acc, host["sample_id"], st)
        sel = _sample_rows(host["sample_id"].numpy(), host["student"].shape[0], rng)
        stats.append(st)
        picks.append(sel)
        subs.append({k: v[torch.as_tensor(sel)].clone() for k, v in host.items()})
        del ch, host
    _ORACLE_CACHE[wl.name] = (stats, picks, subs, acc)
    return _ORACLE_CACHE[wl.name]


def _shard_cuts(wl, parts):
    per = 8 if wl.dtype == torch.bfloat16 else 4  # columns per 16 bytes
    return [0] + [per * ((wl.V * k // parts) // per) for k in range(1, parts)] + [wl.V]


def _shards(ch, cuts):
    return [(a, fb.Chunk(ch["student"][:, a:b], ch["teacher"][:, a:b], ch["behav_logprob"], ch["tokens"], ch["mask"],
                         ch["sample_id"])) for a, b in zip(cuts[:-1], cuts[1:])]


def _run_full_size(wl, use_row_ws, vocab_parts=0):
    """vocab_parts > 1: the same comparison through the vocabulary-sharded entry points, all
    holders played in turn on the one GPU."""
    P = par.PARAMS
    p = fb.params(**P)
    B = wl.B
    stats_o, picks, subs, acc_o = _oracle_measurement(wl)
    fr = orc.sample_freshness(acc_o, wl.tau, wl.H, None, P["alpha"], P["beta"], P["xi"])
    loss_o, per_o = orc.loss(fr, P["lam"])
    buf = pl.BatchBuffers(B, DEV)
    tau = torch.as_tensor(wl.tau, device=DEV)
    H = torch.as_tensor(wl.H, device=DEV)
    rows_out = []
    worst = dict(lp=0.0, kl=0.0, ratio=0.0, f=0.0, loss=0.0, grad_abs=0.0, grad_rel=0.0, rowsum=0.0)

    # ---- measurement phase, chunk by chunk: every per-row output of every row against the oracle
    for j in range(wl.n_chunks):
        ch = synth.gen_chunk(wl, j, DEV)
        r = pl.RowOutputs.alloc(ch["student"].shape[0], DEV)
        if vocab_parts > 1:
            shards = _shards(ch, _shard_cuts(wl, vocab_parts))
            parts = torch.empty((len(shards), ch["tokens"].numel(), 8), dtype=torch.float32, device=DEV)
            for k, (a, sh) in enumerate(shards):
                fb.fopd_shard_stats(sh, a, wl.V, parts[k])
            fb.fopd_shard_merge(parts, ch["behav_logprob"], ch["tokens"], ch["mask"], ch["sample_id"], wl.V, B,
                                buf.acc, r.row_ws, lp_s=r.lp_s, lp_t=r.lp_t, kl=r.kl, ratio=r.ratio,
                                status=buf.status)
        else:
            pl.measure([pl.to_chunk(ch)], buf, [r], keep_row_ws=True)
        st = stats_o[j]
        g = {k: getattr(r, k).cpu().numpy().astype(np.float64) for k in ("lp_s", "lp_t", "kl", "ratio")}
        valid = st.valid.astype(bool)
        for k in g:
            assert np.all(g[k][~valid] == 0.0), k
        if valid.any():
            worst["lp"] = max(worst["lp"], np.abs(g["lp_s"] - st.lp_s)[valid].max(),
                              np.abs(g["lp_t"] - st.lp_t)[valid].max())
            worst["kl"] = max(worst["kl"], (np.abs(g["kl"] - st.kl) / np.maximum(1.0, st.kl))[valid].max())
            worst["ratio"] = max(worst["ratio"], (np.abs(g["ratio"] - st.rho)[valid] / st.rho[valid]).max())
        rows_out.append(r)
        del ch
    assert worst["lp"] <= par.TOL_LOGPROB and worst["kl"] <= 1e-4 and worst["ratio"] <= 1.1 * par.TOL_LOGPROB, worst

    # ---- per-sample sums: counts exact against the oracle; and (a property that holds at any
    # size) equal to the fp64 sums of the per-row outputs in any order
    acc = buf.acc.cpu().numpy()
    assert np.array_equal(acc[:, 0], acc_o[:, 0]), "aligned-row counts differ"
    want = np.zeros((B, 3))
    for j, r in enumerate(rows_out):
        lo, hi = wl.chunk_range(j)
        ws = r.row_ws.cpu().numpy().astype(np.float64)
        sid, m = wl.sample_id[lo:hi], wl.mask[lo:hi].astype(bool)
        d = ws[m, 3]
        np.add.at(want[:, 0], sid[m], 1.0)
        np.add.at(want[:, 1], sid[m], np.exp(d) * d - np.expm1(d))
        np.add.at(want[:, 2], sid[m], ws[m, 2])
    assert np.allclose(acc[:, :3], want, rtol=1e-9, atol=1e-12)
    assert np.array_equal(acc[:, 3], np.bincount(wl.sample_id, minlength=B).astype(np.float64))

    # ---- freshness, gate, weights against the oracle's own sums
    pl.freshness(buf, tau, H, None, p)
    ok = fr.valid.astype(bool)
    rel = lambda a, b: (np.abs(a - b) / np.maximum(np.abs(b), 1e-2))[ok].max() if ok.any() else 0.0
    get = lambda name: getattr(buf, name).cpu().numpy().astype(np.float64)
    for name in ("f", "w", "d_roll", "l_distill", "m_align", "coef"):
        assert np.all(get(name)[~ok] == 0.0), name
    worst["f"] = max(rel(get("f"), fr.f), rel(get("d_roll"), fr.D_roll), rel(get("l_distill"), fr.ell),
                     rel(get("m_align"), fr.m))
    assert worst["f"] <= par.TOL_REL, worst
    assert (np.abs(get("w") - fr.w)[ok] <= par.TOL_REL * fr.f[ok]).all()
    decided = np.abs(fr.f - P["xi"]) > 1e-5
    assert decided[ok].all(), "a sample sits on the gate threshold: pick another seed"
    assert np.array_equal(get("w") > 0, fr.w > 0)
    assert (np.abs(get("coef") - fr.coef)[ok] <= par.TOL_REL * fr.f[ok] / (B * np.maximum(acc_o[ok, 0], 1))).all()
    coef = fr.coef  # the oracle's weights: nothing below takes an input from the CUDA path

    # ---- optimisation phase, chunk by chunk (chunks regenerated from their seeds)
    for j in range(wl.n_chunks):
        ch = synth.gen_chunk(wl, j, DEV)
        dl = torch.full_like(ch["student"], float("nan"))
        if vocab_parts > 1:
            for k, (a, sh) in enumerate(_shards(ch, _shard_cuts(wl, vocab_parts))):
                fb.fopd_shard_loss_fwd_bwd(sh, a, wl.V, B, buf.coef, rows_out[j].row_ws, p,
                                           dl[:, a:a + sh.student.shape[1]], loss_acc=buf.loss_acc if k == 0 else None)
        else:
            fb.fopd_loss_fwd_bwd(pl.to_chunk(ch), B, buf.coef, p, dl, buf.loss_acc,
                                 row_ws=rows_out[j].row_ws if use_row_ws else None, status=buf.status)
        lo, hi = wl.chunk_range(j)
        active = torch.as_tensor((wl.mask[lo:hi] > 0) & (coef[wl.sample_id[lo:hi]] > 0), device=DEV)
        if (~active).any():
            z = dl[~active]
            assert float(z.abs().max()) == 0.0 and not bool(torch.signbit(z).any())
        if active.any():
            a = dl if bool(active.all()) else dl[active]
            rs = torch.zeros(a.shape[0], dtype=torch.float64, device=DEV)
            l1 = torch.zeros_like(rs)
            for c0 in range(0, a.shape[1], 8192):  # column blocks keep the fp64 temporaries small
                blk = a[:, c0:c0 + 8192].double()
                rs += blk.sum(1)
                l1 += blk.abs().sum(1)
            excess = (rs.abs() - par.out_ulp(dl.dtype) * l1).clamp_min(0.0).max()
            worst["rowsum"] = max(worst["rowsum"], float(excess) / float(coef.max()))
        sel, sub, st = picks[j], subs[j], stats_o[j]
        g_ref = orc.grad_rows(sub["student"], sub["teacher"], sub["tokens"], sub["behav_logprob"], sub["mask"],
                              sub["sample_id"], coef, P["lam"], np.arange(len(sel)))
        g_gpu = dl[torch.as_tensor(sel, device=DEV)].double().cpu().numpy()
        err = np.abs(g_gpu - g_ref)
        worst["grad_abs"] = max(worst["grad_abs"], float(err.max()))
        cf = coef[np.clip(sub["sample_id"].numpy(), 0, B - 1)] * st.valid[sel]
        cp = cf[:, None] * np.exp(sub["student"].double().numpy() - st.lse_s[sel, None])
        bound = (par.out_ulp(dl.dtype) + 2e-5) * np.abs(g_ref) + 2e-5 * cp + 1e-30
        ycol = np.clip(sub["tokens"].numpy(), 0, wl.V - 1)
        bound[np.arange(len(sel)), ycol] += 1e-5 * np.abs(cf * P["lam"] * st.rho[sel] * (1 + np.abs(st.d[sel])))
        worst["grad_rel"] = max(worst["grad_rel"], float((err / bound).max()))
        del ch, dl
    fb.fopd_loss_finalize(buf.loss_acc, buf.acc, buf.w, B, p, buf.loss, per_sample_loss=buf.per_sample_loss)
    assert fb.fopd_check_status(buf.status) == 0
    assert worst["grad_abs"] <= par.TOL_GRAD_ABS and worst["grad_rel"] <= 1.0 and worst["rowsum"] <= 1e-5, worst

    # ---- loss (Eq. 16) against the oracle
    got = float(buf.loss.cpu()[0])
    worst["loss"] = abs(got - loss_o) / max(abs(loss_o), 1e-2)
    assert worst["loss"] <= par.TOL_REL, (got, loss_o)
    per_gpu = buf.per_sample_loss.cpu().numpy().astype(np.float64)
    assert (np.abs(per_gpu - per_o) <= par.TOL_REL * np.maximum(np.abs(per_o), 1e-2)).all()
    return worst


@pytest.mark.parametrize("use_row_ws", [True, False], ids=["cached", "on_chip"])
def test_reasoning_full_size(use_row_ws):
    wl = synth.reasoning()  # 32,768 x 151,936 bf16: the workload bench.py times
    print(wl.name, wl.n_rows, wl.V, _run_full_size(wl, use_row_ws))


def test_reasoning_full_size_vocab_sharded():
    wl = synth.reasoning()  # eight holders of 18,992 columns each, row pitch 151,936
    print(wl.name, wl.n_rows, wl.V, _run_full_size(wl, True, vocab_parts=8))


def test_reasoning_full_size_from_host_buffers():
    """fopd_step_host on the benchmark workload: per-sample outputs and the loss against the
    oracle's measurement over every row, the gradient on the oracle's sampled rows, zeros on
    every row that is not differentiated."""
    wl = synth.reasoning()
    P = par.PARAMS
    stats_o, picks, subs, acc_o = _oracle_measurement(wl)
    fr = orc.sample_freshness(acc_o, wl.tau, wl.H, None, P["alpha"], P["beta"], P["xi"])
    loss_o, per_o = orc.loss(fr, P["lam"])
    host = [{k: v.cpu().pin_memory() for k, v in synth.gen_chunk(wl, j, DEV).items()} for j in range(wl.n_chunks)]
    hchunks = [pl.to_chunk(c) for c in host]
    dl = [torch.full_like(c["student"], float("nan")).pin_memory() for c in host]
    ws = torch.empty(fb.fopd_step_host_workspace_bytes(hchunks, wl.B, True), dtype=torch.uint8, device=DEV)
    res = fb.fopd_step_host(hchunks, wl.B, torch.as_tensor(wl.tau), torch.as_tensor(wl.H), None, fb.params(**P), dl,
                            ws)
    assert int(res["status_bits"][0]) == 0
    ok = fr.valid.astype(bool)
    rel = lambda a, b: (np.abs(a.numpy().astype(np.float64) - b) / np.maximum(np.abs(b), 1e-2))[ok].max()
    assert max(rel(res["f"], fr.f), rel(res["d_roll"], fr.D_roll), rel(res["l_distill"], fr.ell),
               rel(res["m_align"], fr.m), rel(res["w"], fr.w)) <= par.TOL_REL
    assert abs(float(res["loss"][0]) - loss_o) <= par.TOL_REL * max(abs(loss_o), 1e-2)
    assert (np.abs(res["per_sample_loss"].numpy() - per_o) <= par.TOL_REL * np.maximum(np.abs(per_o), 1e-2)).all()
    for j, c in enumerate(host):
        lo, hi = wl.chunk_range(j)
        active = torch.as_tensor((wl.mask[lo:hi] > 0) & (fr.coef[wl.sample_id[lo:hi]] > 0))
        z = dl[j][~active].view(torch.int16)  # +0 exactly: all bits clear
        assert int(z.abs().max()) == 0
        sel, sub = picks[j], subs[j]
        g_ref = orc.grad_rows(sub["student"], sub["teacher"], sub["tokens"], sub["behav_logprob"], sub["mask"],
                              sub["sample_id"], fr.coef, P["lam"], np.arange(len(sel)))
        g = dl[j][torch.as_tensor(sel)].double().numpy()
        assert np.isfinite(g).all() and np.abs(g - g_ref).max() <= par.TOL_GRAD_ABS
        assert bool(torch.isfinite(dl[j]).all()), "a gradient row was never written"


@pytest.mark.parametrize("name,use_row_ws", [("tool_use", True), ("tool_use", False), ("coding_agent", False),
                                             ("coding_agent", True)])
def test_chunked_workloads_full_size(name, use_row_ws):
    wl = synth.WORKLOADS[name]()  # 16,384-row chunks cutting across samples, V = 151,936
    print(wl.name, wl.n_rows, wl.V, wl.n_chunks, _run_full_size(wl, use_row_ws))


@pytest.mark.parametrize("rows,V,use_row_ws", [(4096, 32000, False), (16384, 128256, True), (65536, 151936, False),
                                               (4096, 151936, False), (65536, 32000, True), (16384, 151936, True)])
def test_roofline_points_full_size(rows, V, use_row_ws):
    wl = synth.roofline_point(rows, V)
    print(wl.name, _run_full_size(wl, use_row_ws))
