"""GPU parity of the diagnostic entry points (supervision drift of Eq. 10, response
entropy, buffer refresh rule of Eq. 14-15) against the fp64 CPU oracle."""
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


def _divergence(first, second, mask, sid, B, vocab=None):
    n = first.shape[0]
    acc = torch.zeros((B, 3), dtype=torch.float64, device=DEV)
    kl = torch.full((n,), 7.0, device=DEV)
    ent = torch.full((n,), 7.0, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    fb.fopd_row_divergence(first, second, mask, sid, B, acc, kl=kl, entropy=ent, vocab=vocab, status=status)
    return kl.cpu().numpy().astype(np.float64), ent.cpu().numpy().astype(np.float64), acc, int(status.cpu()[0])


@pytest.mark.parametrize("name", ["tool_use", "coding_agent"])
def test_supervision_drift_against_oracle(name):
    """Teacher under the current context vs the stored one (here: teacher logits and a
    perturbed copy), on the supervision-aligned positions, chunk by chunk."""
    wl = synth.WORKLOADS[name](scale=1 / 16)
    B = wl.B
    acc = torch.zeros((B, 3), dtype=torch.float64, device=DEV)
    rng = np.random.default_rng(5)
    sup_mask_all = (wl.mask & (rng.random(wl.n_rows) > 0.3)).astype(np.uint8)  # U^sup differs from U^roll
    sup_mask_all[wl.sample_id == 2] = 0                                          # one sample with U^sup empty
    kl_ref, ent_ref = [], []
    for j in range(wl.n_chunks):
        ch = synth.gen_chunk(wl, j, DEV)
        lo, hi = wl.chunk_range(j)
        g = torch.Generator(device=DEV).manual_seed(100 + j)
        cur = ch["teacher"]
        old = (cur.float() + 0.4 * torch.randn(cur.shape, generator=g, device=DEV)).to(cur.dtype)
        m = torch.as_tensor(sup_mask_all[lo:hi], device=DEV)
        n = cur.shape[0]
        kl = torch.full((n,), 7.0, device=DEV)
        ent = torch.full((n,), 7.0, device=DEV)
        fb.fopd_row_divergence(cur, old, m, ch["sample_id"], B, acc, kl=kl, entropy=ent)
        k_o, e_o = orc.row_divergence(cur.cpu(), old.cpu(), sup_mask_all[lo:hi])
        mb = sup_mask_all[lo:hi].astype(bool)
        k_g, e_g = kl.cpu().numpy().astype(np.float64), ent.cpu().numpy().astype(np.float64)
        assert np.all(k_g[~mb] == 0) and np.all(e_g[~mb] == 0)
        if mb.any():  # a chunk may lie entirely inside the sample whose set was emptied
            assert np.abs(k_g - k_o)[mb].max() <= 1e-4 * max(1.0, k_o.max())
            assert np.abs(e_g - e_o)[mb].max() <= par.TOL_LOGPROB
        kl_ref.append(k_o)
        ent_ref.append(e_o)
    d_o, m_o, e_o, cnt_o = orc.supervision_drift(np.concatenate(kl_ref), np.concatenate(ent_ref), sup_mask_all,
                                                 wl.sample_id, wl.H, B)
    d = torch.empty(B, device=DEV); m = torch.empty(B, device=DEV); e = torch.empty(B, device=DEV)
    fb.fopd_supervision_drift(acc, torch.as_tensor(wl.H, device=DEV), B, d_sup=d, m_sup=m, mean_entropy=e)
    assert np.array_equal(acc[:, 0].cpu().numpy(), cnt_o)  # counts exact
    dg = d.cpu().numpy().astype(np.float64)
    fin = np.isfinite(d_o)
    assert np.array_equal(np.isinf(dg), ~fin) and not fin[2]
    assert np.allclose(dg[fin], d_o[fin], rtol=par.TOL_REL, atol=1e-6)
    assert np.allclose(m.cpu().numpy(), m_o, rtol=1e-6) and np.allclose(e.cpu().numpy(), e_o, rtol=par.TOL_REL)

    # freshness with this D_sup: the sample without supervision positions is invalid (Algorithm 1)
    # (the oracle's D_sup goes to both sides: no oracle input comes from the CUDA path)
    chunks = [synth.gen_chunk(wl, j, DEV) for j in range(wl.n_chunks)]
    out = par.compare(chunks, B, wl.tau, wl.H, d_sup=d_o.astype(np.float32), grad_rows_per_chunk=8)
    buf, *_ = par.gpu_run(chunks, B, wl.tau, wl.H, d_sup=d_o.astype(np.float32))
    assert float(buf.f[2]) == 0 and float(buf.w[2]) == 0 and float(buf.coef[2]) == 0 and float(buf.m_align[2]) == 0
    print(name, out)


@pytest.mark.parametrize("V,stride,dtype", [(5, 8, torch.bfloat16), (33, 40, torch.float32), (4099, 4104, torch.bfloat16),
                                            (151936, 151936, torch.bfloat16)])
def test_row_divergence_shapes_entropy_and_student_teacher_kl(V, stride, dtype):
    rng = np.random.RandomState(V)
    B, n = 2, 21
    sid = np.repeat(np.arange(B, dtype=np.int32), [9, 12])
    mask = (rng.rand(n) > 0.25).astype(np.uint8)
    wl = synth.Workload("div", B, V, dtype, n, sid, mask, np.zeros(B, np.int32), np.array([9, 12], np.int32), seed=V % 911)
    ch = synth.gen_chunk(wl, 0, DEV, row_block=8, row_stride=stride)
    ch["student"][:, V:] = 1e4   # pitch padding must not be read
    ch["teacher"][:, V:] = -1e4
    k_g, e_g, acc, bits = _divergence(ch["student"], ch["teacher"], ch["mask"], ch["sample_id"], B, vocab=V)
    k_o, e_o = orc.row_divergence(ch["student"][:, :V].cpu().contiguous(), ch["teacher"][:, :V].cpu().contiguous(), mask)
    mb = mask.astype(bool)
    assert bits == 0 and np.all(k_g[~mb] == 0) and np.all(e_g[~mb] == 0)
    assert np.abs(k_g - k_o).max() <= 1e-4 * max(1.0, k_o.max()) and np.abs(e_g - e_o).max() <= par.TOL_LOGPROB
    # same quantity as the token loss of the statistics entry point
    buf = pl.BatchBuffers(B, DEV)
    rows = pl.RowOutputs.alloc(n, DEV)
    pl.measure([pl.to_chunk(ch, V)], buf, [rows])
    assert np.abs(rows.kl.cpu().numpy() - k_g).max() <= 2e-6 * max(1.0, k_o.max())
    a = acc.cpu().numpy()
    assert np.array_equal(a[:, 0], np.bincount(sid[mb], minlength=B))
    assert np.allclose(a[:, 1], np.bincount(sid, weights=k_g, minlength=B), rtol=1e-9)
    # identical tensors: KL exactly zero
    k0, _, _, _ = _divergence(ch["student"], ch["student"], ch["mask"], ch["sample_id"], B, vocab=V)
    assert np.all(k0 == 0.0)
    # a bad sample id is reported and the row treated as masked
    bad = ch["sample_id"].clone(); bad[-1] = B
    k_b, _, _, bits = _divergence(ch["student"], ch["teacher"], torch.ones_like(ch["mask"]), bad, B, vocab=V)
    assert bits == 2 and k_b[-1] == 0.0


@pytest.mark.parametrize("offset,dtype", [(200.0, torch.bfloat16), (-300.0, torch.bfloat16), (100.0, torch.float32),
                                          (-1000.0, torch.float32)])
def test_row_divergence_with_large_logit_offsets(offset, dtype):
    """KL and entropy are shift invariant: logits far from zero (both tensors shifted, and the
    second shifted by a further 50) must give the oracle's values on the same shifted bits."""
    wl = synth.tiny(scale=1 / 8) if dtype == torch.float32 else synth.reasoning(scale=1 / 32)
    ch = synth.gen_chunk(wl, 0, DEV)
    first = (ch["student"].float() + offset).to(dtype)
    second = (ch["teacher"].float() + offset + 50.0).to(dtype)
    lo, hi = wl.chunk_range(0)
    mask = wl.mask[lo:hi]
    k_g, e_g, acc, bits = _divergence(first, second, ch["mask"], ch["sample_id"], wl.B)
    k_o, e_o = orc.row_divergence(first.cpu(), second.cpu(), mask)
    mb = mask.astype(bool)
    assert bits == 0 and mb.any()
    assert np.abs(k_g - k_o)[mb].max() <= 1e-4 * max(1.0, k_o.max())
    assert np.abs(e_g - e_o)[mb].max() <= 1e-4 * max(1.0, e_o.max())
    print(offset, np.abs(k_g - k_o)[mb].max(), np.abs(e_g - e_o)[mb].max())


def test_refresh_decision_against_oracle():
    rng = np.random.default_rng(3)
    cases = []
    f = np.array([0.5, 0.25, 0.75], np.float32); m = np.array([0.5, 1.0, 0.75], np.float32)
    ms = np.array([0.25, 0.25, 0.25], np.float32)
    for kf, kr, ks, since in [(0.4, 0.7, 0.2, 500), (0.5, 0.7, 0.2, 500), (0.4, 0.75, 0.25, 500), (0.4, 0.76, 0.2, 500),
                              (0.4, 0.7, 0.26, 500), (0.6, 0.8, 0.3, 200), (0.6, 0.7, 0.2, 199)]:
        cases.append((f, m, ms, kf, kr, ks, since))
    cases.append((f, m, None, 0.4, 0.7, 0.76, 500))
    for _ in range(20):
        B = int(rng.integers(1, 600))
        cases.append((rng.random(B).astype(np.float32), rng.random(B).astype(np.float32),
                      rng.random(B).astype(np.float32), float(rng.random()), float(rng.random()), float(rng.random()),
                      int(rng.integers(0, 400))))
    for f, m, ms, kf, kr, ks, since in cases:
        B = len(f)
        means = torch.zeros(3, device=DEV); dec = torch.full((2,), -1, dtype=torch.int32, device=DEV)
        fb.fopd_refresh_decision(torch.as_tensor(f, device=DEV), torch.as_tensor(m, device=DEV),
                                 None if ms is None else torch.as_tensor(ms, device=DEV), B, kf, kr, ks, since, 200,
                                 dec, means=means)
        mo, bits, go = orc.refresh_decision(f, m, ms, np.float32(kf), np.float32(kr), np.float32(ks), since, 200)
        assert np.allclose(means.cpu().numpy(), mo, rtol=1e-6)
        decided = np.abs(mo - np.array([kf, kr, ks])) > 1e-6  # the seeded random cases are never at a threshold
        assert decided.all() or B == 3
        assert dec.cpu().tolist() == [bits, int(go)], (kf, kr, ks, since, mo)
