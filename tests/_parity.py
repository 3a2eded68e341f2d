"""Shared machinery of the GPU parity tests: run the CUDA library and the fp64
CPU oracle on the same seeded inputs and compare element by element.

Tolerances (stated for the path: bf16 or fp32 logits, fp32 accumulation):
  |delta logprob| <= 1e-3;  per-sample freshness and loss relative error <= 1e-4;
  dlogits max-abs error <= 1e-5;  gather indices, counts and mask handling
  bit-exact.  On top of those, dlogits is held to a relative bound against the
  oracle value (half a unit in the last place of the output dtype plus the fp32
  evaluation error, which scales with coef * p_s(v)) because the absolute bound
  alone is loose when per-token weights are ~1e-5; grad_rel reports error / bound.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import fopd_oracle as orc
from paper_2605_17862_b200 import binding as fb
from paper_2605_17862_b200 import pipeline as pl

TOL_LOGPROB = 1e-3
TOL_REL = 1e-4
TOL_GRAD_ABS = 1e-5
from paper_2605_17862_b200 import synth

# The library takes alpha, beta, xi, lambda as C floats: both sides get the fp32-rounded values.
PARAMS = synth.f32_params()


def exact(params):
    """Any parameter dict (e.g. ``dict(PARAMS, xi=0.05)``) rounded to fp32 for both sides."""
    return synth.f32_params(**params)


def host_chunk(d):
    return {k: v.detach().cpu() for k, v in d.items()}


def gpu_run(chunks_dev, B, tau, H, d_sup=None, params=PARAMS, use_row_ws=True, vocab=None, want_rows=True,
            loss_kind=0):
    dev = chunks_dev[0]["student"].device
    params = exact(params)
    chunks = [pl.to_chunk(c, vocab, loss_kind) for c in chunks_dev]
    buf = pl.BatchBuffers(B, dev)
    rows = [pl.RowOutputs.alloc(c["student"].shape[0], dev) for c in chunks_dev]
    dlogits = [torch.full_like(c["student"], float("nan")) for c in chunks_dev]
    p = fb.params(**params)
    tau_d = torch.as_tensor(np.asarray(tau, dtype=np.int32), device=dev)
    H_d = torch.as_tensor(np.asarray(H, dtype=np.int32), device=dev)
    ds_d = None if d_sup is None else torch.as_tensor(np.asarray(d_sup, dtype=np.float32), device=dev)
    pl.step(chunks, dlogits, buf, tau_d, H_d, ds_d, p, rows if (want_rows or use_row_ws) else None,
            use_row_ws=use_row_ws)
    bits = fb.fopd_check_status(buf.status)
    return buf, rows, dlogits, bits


def oracle_run(chunks_host, B, tau, H, d_sup=None, params=PARAMS, loss_kind=0):
    params = exact(params)
    return orc.run_batch(chunks_host, B, tau, H, d_sup, params["alpha"], params["beta"], params["xi"], params["lam"],
                         loss_kind)


def out_ulp(dtype):
    """Largest relative rounding error of one store in the output dtype."""
    return 2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -24


def gpu_run_vocab_sharded(cuts):
    """A runner with gpu_run's signature that splits the vocabulary at ``cuts`` (column
    indices, first 0, last V) and plays every holder in turn on the one GPU: all holders'
    partial sums first, then each holder's whole step with the exchange replaced by the
    stack of those partial sums.  Every holder must arrive at bit-identical row statistics,
    sums, freshness and loss; the gradient is assembled from the holders' column ranges."""
    def run(chunks_dev, B, tau, H, d_sup=None, params=PARAMS, use_row_ws=True, vocab=None, want_rows=True):
        dev = chunks_dev[0]["student"].device
        V = vocab or chunks_dev[0]["student"].shape[1]
        assert cuts[0] == 0 and cuts[-1] == V
        params = exact(params)
        p = fb.params(**params)
        tau_d = torch.as_tensor(np.asarray(tau, dtype=np.int32), device=dev)
        H_d = torch.as_tensor(np.asarray(H, dtype=np.int32), device=dev)
        ds_d = None if d_sup is None else torch.as_tensor(np.asarray(d_sup, dtype=np.float32), device=dev)
        dlogits = [torch.full_like(c["student"], float("nan")) for c in chunks_dev]
        ranges = list(zip(cuts[:-1], cuts[1:]))

        def shard(c, a, b):
            return fb.Chunk(c["student"][:, a:b], c["teacher"][:, a:b], c["behav_logprob"], c["tokens"], c["mask"],
                            c["sample_id"])

        parts = []
        for c in chunks_dev:
            n = c["tokens"].numel()
            stack = torch.empty((len(ranges), n, 8), dtype=torch.float32, device=dev)
            for k, (a, b) in enumerate(ranges):
                fb.fopd_shard_stats(shard(c, a, b), a, V, stack[k])
            parts.append(stack)
        results = []
        for k, (a, b) in enumerate(ranges):
            buf = pl.BatchBuffers(B, dev)
            rows = [pl.RowOutputs.alloc(c["student"].shape[0], dev) for c in chunks_dev]
            it = iter(parts)
            own = []

            def gather(part, it=it, k=k, own=own):
                stack = next(it)
                assert torch.equal(part, stack[k])  # this holder's own sums are reproducible
                return stack

            pl.step_vocab_sharded([shard(c, a, b) for c in chunks_dev], a, V, [d[:, a:b] for d in dlogits], buf,
                                  tau_d, H_d, ds_d, p, rows, gather=gather)
            results.append((buf, rows))
        buf0, rows0 = results[0]
        for buf, rows in results[1:]:
            for name in ("acc", "loss_acc", "f", "w", "coef", "loss", "per_sample_loss", "status"):
                assert torch.equal(getattr(buf, name), getattr(buf0, name)), name
            for r, r0 in zip(rows, rows0):
                assert torch.equal(r.row_ws, r0.row_ws) and torch.equal(r.lp_s, r0.lp_s)
        return buf0, rows0, dlogits, fb.fopd_check_status(buf0.status)
    return run


def compare(chunks_dev, B, tau, H, d_sup=None, params=PARAMS, use_row_ws=True, grad_rows_per_chunk=None,
            seed=0, expect_bits=0, vocab=None, runner=None, loss_kind=0):
    """Full comparison of one batch; returns a dict of the maxima seen.  loss_kind 1: the
    sampled-token form of the token loss (the oracle's per-token loss then stands in its kl field)."""
    params = exact(params)
    if loss_kind:
        assert runner is None
        buf, rows, dlogits, bits = gpu_run(chunks_dev, B, tau, H, d_sup, params, use_row_ws, vocab, loss_kind=loss_kind)
    else:
        buf, rows, dlogits, bits = (runner or gpu_run)(chunks_dev, B, tau, H, d_sup, params, use_row_ws, vocab)
    assert bits == expect_bits, f"device status bits {bits}"
    V = vocab or chunks_dev[0]["student"].shape[1]
    hc = [host_chunk(c) for c in chunks_dev]
    if vocab:
        for c in hc:
            c["student"] = c["student"][:, :V].contiguous()
            c["teacher"] = c["teacher"][:, :V].contiguous()
    ref = oracle_run(hc, B, tau, H, d_sup, params, loss_kind)
    out = dict(lp=0.0, kl=0.0, ratio=0.0, f=0.0, loss=0.0, grad_abs=0.0, grad_rel=0.0, rowsum=0.0, grad_max=0.0)

    # ---- per-token outputs
    for j, st in enumerate(ref.stats):
        r = rows[j]
        valid = st.valid.astype(bool)
        g = {k: getattr(r, k).cpu().numpy().astype(np.float64) for k in ("lp_s", "lp_t", "kl", "ratio")}
        ws = r.row_ws.cpu().numpy().astype(np.float64) if use_row_ws else None  # not written otherwise
        for k in g:  # mask handling is exact: not-aligned rows are exactly zero
            assert np.all(g[k][~valid] == 0.0), k
        if use_row_ws:
            assert np.all(ws[~valid] == 0.0)
        if valid.any():
            out["lp"] = max(out["lp"], np.abs(g["lp_s"] - st.lp_s)[valid].max(), np.abs(g["lp_t"] - st.lp_t)[valid].max())
            if use_row_ws:
                out["lp"] = max(out["lp"], np.abs(ws[:, 0] - st.lse_s)[valid].max(), np.abs(ws[:, 1] - st.lse_t)[valid].max())
            out["kl"] = max(out["kl"], (np.abs(g["kl"] - st.kl) / np.maximum(1.0, np.abs(st.kl)))[valid].max())
            out["ratio"] = max(out["ratio"], (np.abs(g["ratio"] - st.rho)[valid] / st.rho[valid]).max())
    assert out["lp"] <= TOL_LOGPROB, out
    assert out["kl"] <= 1e-4, out
    assert out["ratio"] <= 1.1 * TOL_LOGPROB, out

    # ---- per-sample sums, freshness, gate
    acc = buf.acc.cpu().numpy()
    assert np.array_equal(acc[:, 0], ref.acc[:, 0]), "aligned-row counts differ"
    fr = ref.fresh
    f = buf.f.cpu().numpy().astype(np.float64)
    w = buf.w.cpu().numpy().astype(np.float64)
    inval = ~fr.valid.astype(bool)
    for name in ("f", "w", "m_align", "coef", "d_roll", "l_distill"):
        assert np.all(getattr(buf, name).cpu().numpy()[inval] == 0.0), name
    ok = fr.valid.astype(bool)
    if ok.any():
        # relative error, with an absolute floor because D_roll and the mean KL inherit the
        # ~1e-6 absolute fp32 error of the per-row values when they are themselves near zero
        rel = lambda a, b: (np.abs(a - b) / np.maximum(np.abs(b), 1e-2))[ok].max()
        out["f"] = max(rel(f, fr.f), rel(buf.d_roll.cpu().numpy(), fr.D_roll), rel(buf.l_distill.cpu().numpy(), fr.ell),
                       rel(buf.m_align.cpu().numpy(), fr.m))
        assert out["f"] <= TOL_REL, out
        assert (np.abs(w - fr.w)[ok] <= TOL_REL * fr.f[ok]).all()
        decided = np.abs(fr.f - params["xi"]) > 1e-5  # gate decisions away from the threshold agree
        assert np.array_equal((w > 0)[ok & decided], (fr.w > 0)[ok & decided])
        cf = buf.coef.cpu().numpy().astype(np.float64)
        assert (np.abs(cf - fr.coef)[ok] <= TOL_REL * fr.f[ok] / (B * np.maximum(ref.acc[ok, 0], 1))).all()
    means = buf.buffer_means.cpu().numpy()
    assert abs(means[0] - fr.f.mean()) <= TOL_REL * max(fr.f.mean(), 1e-30) + 1e-12
    assert abs(means[1] - fr.m.mean()) <= TOL_REL * max(fr.m.mean(), 1e-30) + 1e-12

    # ---- loss
    loss = float(buf.loss.cpu()[0])
    out["loss"] = abs(loss - ref.loss) / max(abs(ref.loss), 1e-2)
    assert out["loss"] <= TOL_REL, (loss, ref.loss)
    per = buf.per_sample_loss.cpu().numpy().astype(np.float64)
    assert (np.abs(per - ref.per_sample_loss) <= TOL_REL * np.maximum(np.abs(ref.per_sample_loss), 1e-2)).all()

    # ---- gradient
    rng = np.random.default_rng(seed)
    for j, c in enumerate(hc):
        n = c["student"].shape[0]
        if n == 0:
            continue
        dl = dlogits[j]
        active_dev = torch.as_tensor(ref.stats[j].valid.astype(bool) &
                                     (fr.coef[np.clip(c["sample_id"].numpy(), 0, B - 1)] > 0), device=dl.device)
        # exact zeros on every row that is masked, padded, bad or gated (whole tensor, on device)
        if (~active_dev).any():
            assert float(dl[~active_dev][:, :V].abs().max()) == 0.0
            assert not bool(torch.signbit(dl[~active_dev][:, :V]).any())
        # every active row sums to ~0 (both terms are tangent to the simplex)
        if active_dev.any():
            act = dl[active_dev][:, :V].double()
            rs, l1 = act.sum(1).abs(), act.abs().sum(1)
            excess = (rs - out_ulp(dl.dtype) * l1).clamp_min(0.0).max()
            out["rowsum"] = max(out["rowsum"], float(excess) / float(fr.coef.max()))
        if grad_rows_per_chunk is None or grad_rows_per_chunk >= n:
            sel = np.arange(n)
        else:
            must = np.array([0, n - 1])
            sid = c["sample_id"].numpy()
            edges = np.nonzero(np.diff(sid))[0]
            must = np.concatenate([must, edges, edges + 1])
            sel = np.unique(np.concatenate([must, rng.choice(n, size=grad_rows_per_chunk, replace=False)]))
        g_ref = orc.grad_rows(c["student"], c["teacher"], c["tokens"], c["behav_logprob"], c["mask"],
                              c["sample_id"], fr.coef, params["lam"], sel, loss_kind)
        g_gpu = dl[torch.as_tensor(sel, device=dl.device)][:, :V].double().cpu().numpy()
        err = np.abs(g_gpu - g_ref)
        out["grad_abs"] = max(out["grad_abs"], float(err.max()))
        out["grad_max"] = max(out["grad_max"], float(np.abs(g_ref).max()))
        # element-wise bound: output rounding u |g| plus fp32 evaluation error, which scales
        # with coef * p_s(v) (and with coef * lambda * rho * d at the stored token)
        st = ref.stats[j]
        S64 = c["student"][sel][:, :V].double().numpy()
        cf = fr.coef[np.clip(c["sample_id"].numpy()[sel], 0, B - 1)] * st.valid[sel]
        cp = cf[:, None] * np.exp(S64 - st.lse_s[sel, None])
        bound = (out_ulp(dl.dtype) + 2e-5) * np.abs(g_ref) + 2e-5 * cp + 1e-30
        # the gradient is linear in the sample's weight, which has a tolerance of its own (checked
        # above): near the gate w = f - xi loses relative accuracy by cancellation, and that much
        # of the difference belongs to the weight, not to the gradient sweep
        cf_gpu = buf.coef.cpu().numpy().astype(np.float64)
        rel_w = np.where(fr.coef > 0, np.abs(cf_gpu - fr.coef) / np.maximum(fr.coef, 1e-300), 0.0)
        out["w_rel"] = max(out.get("w_rel", 0.0), float(rel_w.max()))
        bound += rel_w[np.clip(c["sample_id"].numpy()[sel], 0, B - 1)][:, None] * np.abs(g_ref)
        ycol = np.clip(c["tokens"].numpy()[sel], 0, V - 1)
        # d = lp_s - b carries the absolute fp32 error of the log-normaliser (~1e-6), so the
        # anchor term lambda * rho * d at the stored token has an absolute, not relative, error
        bound[np.arange(len(sel)), ycol] += 1e-5 * np.abs(cf * params["lam"] * st.rho[sel] * (1 + np.abs(st.d[sel])))
        if loss_kind:
            # the row is weight * (1[v = y] - p_s(v)) with weight = coef rho (r + lambda d); r and d carry
            # the absolute fp32 error of the log-normalisers (~1e-6 each), whatever their own size
            onehot = np.zeros_like(cp)
            onehot[np.arange(len(sel)), ycol] = 1.0
            p_s = np.exp(S64 - st.lse_s[sel, None])
            bound += 1e-5 * np.abs(cf * st.rho[sel])[:, None] * np.abs(onehot - p_s)
        out["grad_rel"] = max(out["grad_rel"], float((err / bound).max()))
    # 1e-5 absolute, unless the rounding of the largest output alone exceeds it (tests with
    # a handful of rows per sample have per-token weights ~1e-2, far above any real batch)
    assert out["grad_abs"] <= max(TOL_GRAD_ABS, 1.01 * out_ulp(chunks_dev[0]["student"].dtype) * out["grad_max"]), out
    # row sums vanish up to output rounding (below ulp * L1 of the row) plus the fp32
    # evaluation error of the row constants, which is absolute at the scale of coef
    assert out["rowsum"] <= 1e-5, out
    assert out["grad_rel"] <= 1.0, out
    return out
