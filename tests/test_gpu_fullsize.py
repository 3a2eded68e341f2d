"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The fp64 CPU oracle cannot sweep tens of gigabytes of logits, so these tests
check (a) every per-row output and the gradient on a seeded sample of rows that
the oracle computes one by one -- always including the first and last row of
every chunk and the rows on both sides of every sample boundary -- and (b)
properties that hold at any size: the per-sample sums equal the fp64 sums of
the per-row outputs (counts exactly), freshness / gate / weights equal the
oracle's formulas applied to those sums, rows that are not differentiated are
exactly +0, every differentiated row of the gradient sums to zero.  Chunks are
streamed (generated, used, freed) exactly as the chunked configurations say.
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


def _run_full_size(wl, use_row_ws):
    P = par.PARAMS
    p = fb.params(**P)
    B = wl.B
    buf = pl.BatchBuffers(B, DEV)
    tau = torch.as_tensor(wl.tau, device=DEV)
    H = torch.as_tensor(wl.H, device=DEV)
    rng = np.random.default_rng(wl.seed)
    rows_out, picks, refs = [], [], []
    worst = dict(lp=0.0, kl=0.0, ratio=0.0, f=0.0, loss=0.0, grad_abs=0.0, grad_rel=0.0, rowsum=0.0)

    # ---- measurement phase, chunk by chunk
    for j in range(wl.n_chunks):
        ch = synth.gen_chunk(wl, j, DEV)
        n = ch["student"].shape[0]
        r = pl.RowOutputs.alloc(n, DEV)
        pl.measure([pl.to_chunk(ch)], buf, [r], keep_row_ws=True)
        sel = _sample_rows(ch["sample_id"].cpu().numpy(), n, rng)
        sub = _sub_chunk(ch, sel)
        st = orc.token_stats(sub["student"], sub["teacher"], sub["tokens"], sub["behav_logprob"], sub["mask"],
                             sub["sample_id"], B)
        g = {k: getattr(r, k)[torch.as_tensor(sel, device=DEV)].cpu().numpy().astype(np.float64)
             for k in ("lp_s", "lp_t", "kl", "ratio")}
        valid = st.valid.astype(bool)
        for k in g:
            assert np.all(g[k][~valid] == 0.0), k
        if valid.any():
            worst["lp"] = max(worst["lp"], np.abs(g["lp_s"] - st.lp_s)[valid].max(),
                              np.abs(g["lp_t"] - st.lp_t)[valid].max())
            worst["kl"] = max(worst["kl"], (np.abs(g["kl"] - st.kl) / np.maximum(1.0, st.kl))[valid].max())
            worst["ratio"] = max(worst["ratio"], (np.abs(g["ratio"] - st.rho)[valid] / st.rho[valid]).max())
        rows_out.append(r)
        picks.append(sel)
        refs.append((sub, st))
        del ch
    assert worst["lp"] <= par.TOL_LOGPROB and worst["kl"] <= 1e-4 and worst["ratio"] <= 1.1 * par.TOL_LOGPROB, worst

    # ---- per-sample sums against fp64 sums of the per-row outputs (any-size property)
    acc = buf.acc.cpu().numpy()
    want = np.zeros((B, 3))
    for j, r in enumerate(rows_out):
        lo, hi = wl.chunk_range(j)
        ws = r.row_ws.cpu().numpy().astype(np.float64)
        sid, m = wl.sample_id[lo:hi], wl.mask[lo:hi].astype(bool)
        d = ws[m, 3]
        np.add.at(want[:, 0], sid[m], 1.0)
        np.add.at(want[:, 1], sid[m], np.exp(d) * d - np.expm1(d))
        np.add.at(want[:, 2], sid[m], ws[m, 2])
    assert np.array_equal(acc[:, 0], want[:, 0]), "aligned-row counts differ"
    assert np.allclose(acc[:, 1:3], want[:, 1:3], rtol=1e-9, atol=1e-12)
    assert np.array_equal(acc[:, 3], np.bincount(wl.sample_id, minlength=B).astype(np.float64))

    # ---- freshness, gate, weights: the oracle's formulas on the same sums
    pl.freshness(buf, tau, H, None, p)
    fr = orc.sample_freshness(np.ascontiguousarray(acc[:, :3]), wl.tau, wl.H, None, P["alpha"], P["beta"], P["xi"])
    ok = fr.valid.astype(bool)
    for name, ref in (("f", fr.f), ("w", fr.w), ("d_roll", fr.D_roll), ("l_distill", fr.ell), ("m_align", fr.m),
                      ("coef", fr.coef)):
        got = getattr(buf, name).cpu().numpy().astype(np.float64)
        assert np.all(got[~ok] == 0.0), name
        assert np.allclose(got[ok], ref[ok], rtol=1e-6, atol=1e-12), name
    coef = buf.coef.cpu().numpy().astype(np.float64)

    # ---- optimisation phase, chunk by chunk (chunks regenerated from their seeds)
    for j in range(wl.n_chunks):
        ch = synth.gen_chunk(wl, j, DEV)
        dl = torch.full_like(ch["student"], float("nan"))
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
        sel = picks[j]
        sub, st = refs[j]
        g_ref = orc.grad_rows(sub["student"], sub["teacher"], sub["tokens"], sub["behav_logprob"], sub["mask"],
                              sub["sample_id"], coef, P["lam"], np.arange(len(sel)))
        g_gpu = dl[torch.as_tensor(sel, device=DEV)].double().cpu().numpy()
        err = np.abs(g_gpu - g_ref)
        worst["grad_abs"] = max(worst["grad_abs"], float(err.max()))
        cf = coef[np.clip(sub["sample_id"].numpy(), 0, B - 1)] * st.valid
        cp = cf[:, None] * np.exp(sub["student"].double().numpy() - st.lse_s[:, None])
        bound = (par.out_ulp(dl.dtype) + 2e-5) * np.abs(g_ref) + 2e-5 * cp + 1e-30
        ycol = np.clip(sub["tokens"].numpy(), 0, wl.V - 1)
        bound[np.arange(len(sel)), ycol] += 1e-5 * np.abs(cf * P["lam"] * st.rho * (1 + np.abs(st.d)))
        worst["grad_rel"] = max(worst["grad_rel"], float((err / bound).max()))
        del ch, dl
    fb.fopd_loss_finalize(buf.loss_acc, buf.acc, buf.w, B, p, buf.loss, per_sample_loss=buf.per_sample_loss)
    assert fb.fopd_check_status(buf.status) == 0
    assert worst["grad_abs"] <= par.TOL_GRAD_ABS and worst["grad_rel"] <= 1.0 and worst["rowsum"] <= 1e-5, worst

    # ---- loss: Eq. 16 from the oracle's per-sample means
    total, per = orc.loss(fr, P["lam"])
    got = float(buf.loss.cpu()[0])
    worst["loss"] = abs(got - total) / max(abs(total), 1e-2)
    assert worst["loss"] <= par.TOL_REL, (got, total)
    per_gpu = buf.per_sample_loss.cpu().numpy().astype(np.float64)
    assert (np.abs(per_gpu - per) <= par.TOL_REL * np.maximum(np.abs(per), 1e-2)).all()
    return worst


@pytest.mark.parametrize("use_row_ws", [True, False], ids=["cached", "on_chip"])
def test_reasoning_full_size(use_row_ws):
    wl = synth.reasoning()  # 32,768 x 151,936 bf16: the workload bench.py times
    print(wl.name, wl.n_rows, wl.V, _run_full_size(wl, use_row_ws))


@pytest.mark.parametrize("name,use_row_ws", [("tool_use", True), ("coding_agent", False)])
def test_chunked_workloads_full_size(name, use_row_ws):
    wl = synth.WORKLOADS[name]()  # 16,384-row chunks cutting across samples, V = 151,936
    print(wl.name, wl.n_rows, wl.V, wl.n_chunks, _run_full_size(wl, use_row_ws))


@pytest.mark.parametrize("rows,V,use_row_ws", [(4096, 32000, False), (16384, 128256, True), (65536, 151936, False)])
def test_roofline_points_full_size(rows, V, use_row_ws):
    wl = synth.roofline_point(rows, V)
    print(wl.name, _run_full_size(wl, use_row_ws))
