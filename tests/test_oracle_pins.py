"""Pins for the fp64 CPU oracle: closed forms, brute force on tiny vocabularies,
float64 library routines, identities and central finite differences.  None of
these re-types the oracle's own formula; each is chosen so that a plausible
slip (a dropped term, a swapped operand, a wrong sign or index) fails it.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import fopd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.json")


def _stats(S, T, y, b, mask=None, sid=None, B=1):
    n = S.shape[0]
    mask = np.ones(n, np.uint8) if mask is None else mask
    sid = np.zeros(n, np.int32) if sid is None else sid
    return orc.token_stats(S, T, y, b, mask, sid, B)


def _rand_rows(rng, n, V, scale=2.0):
    S = (rng.standard_normal((n, V)) * scale).astype(np.float32)
    T = (S + rng.standard_normal((n, V))).astype(np.float32)
    y = rng.integers(0, V, size=n).astype(np.int32)
    b = (-rng.random(n) * 3).astype(np.float32)
    return S, T, y, b


# ----------------------------------------------------------------- lse / logp
def test_lse_brute_force_tiny_vocab():
    rng = np.random.default_rng(0)
    for V in (1, 2, 5, 7, 33):
        S, T, y, b = _rand_rows(rng, 6, V)
        st = _stats(S, T, y, b)
        for n in range(6):
            ref_s = math.log(math.fsum(math.exp(float(z)) for z in S[n]))
            ref_t = math.log(math.fsum(math.exp(float(z)) for z in T[n]))
            assert abs(st.lse_s[n] - ref_s) < 1e-12
            assert abs(st.lse_t[n] - ref_t) < 1e-12
            assert abs(st.lp_s[n] - (float(S[n, y[n]]) - ref_s)) < 1e-12
            assert abs(st.lp_t[n] - (float(T[n, y[n]]) - ref_t)) < 1e-12


def test_lse_shift_invariance_and_constant_row():
    rng = np.random.default_rng(1)
    S, T, y, b = _rand_rows(rng, 4, 50)
    st0 = _stats(S, T, y, b)
    st1 = _stats(S + np.float32(4.0), T - np.float32(2.0), y, b)  # exact shifts in fp32? use powers of two
    # 4.0 and 2.0 shifts of fp32 values are not always exact; compare against widened inputs
    ref_s = torch.logsumexp(torch.from_numpy((S + np.float32(4.0)).astype(np.float64)), 1).numpy()
    assert np.allclose(st1.lse_s, ref_s, atol=1e-12)
    assert np.allclose(st1.lse_s - st0.lse_s, 4.0, atol=1e-5)
    # the KL is unchanged by per-row shifts of either tensor
    assert np.allclose(st1.kl, st0.kl, atol=1e-5)
    V = 37
    C = np.full((1, V), 1.5, np.float32)
    st = _stats(C, C, np.array([3], np.int32), np.array([0.0], np.float32))
    assert abs(st.lse_s[0] - (1.5 + math.log(V))) < 1e-13
    assert abs(st.lp_s[0] + math.log(V)) < 1e-13


def test_logprobs_match_torch_float64_and_sum_to_one():
    rng = np.random.default_rng(2)
    S, T, y, b = _rand_rows(rng, 8, 1000, scale=3.0)
    st = _stats(S, T, y, b)
    ls = torch.log_softmax(torch.from_numpy(S).double(), 1)
    lt = torch.log_softmax(torch.from_numpy(T).double(), 1)
    idx = torch.from_numpy(y.astype(np.int64))[:, None]
    assert np.allclose(st.lp_s, ls.gather(1, idx)[:, 0].numpy(), atol=1e-12)
    assert np.allclose(st.lp_t, lt.gather(1, idx)[:, 0].numpy(), atol=1e-12)
    # exp(S - lse) sums to one: pins the normaliser independently of torch
    p = np.exp(S.astype(np.float64) - st.lse_s[:, None])
    assert np.allclose(p.sum(1), 1.0, atol=1e-12)


def test_bf16_inputs_are_widened_exactly():
    rng = np.random.default_rng(3)
    S32, T32, y, b = _rand_rows(rng, 5, 300, scale=3.0)
    Sb, Tb = torch.from_numpy(S32).bfloat16(), torch.from_numpy(T32).bfloat16()
    st_b = _stats(Sb, Tb, y, b)
    st_f = _stats(Sb.float().numpy(), Tb.float().numpy(), y, b)
    for name in ("lse_s", "lse_t", "lp_s", "lp_t", "kl", "k3"):
        assert np.array_equal(getattr(st_b, name), getattr(st_f, name)), name


# ------------------------------------------------------------------ token KL
def test_kl_zero_when_teacher_equals_student_and_nonnegative():
    rng = np.random.default_rng(4)
    S, T, y, b = _rand_rows(rng, 16, 257)
    st = _stats(S, S.copy(), y, b)
    assert np.all(st.kl == 0.0)  # bitwise zero
    st = _stats(S, S + np.float32(0.5), y, b)
    assert np.all(np.abs(st.kl) < 1e-6)
    st = _stats(S, T, y, b)
    assert np.all(st.kl > 0.0)


def test_kl_bernoulli_closed_form_and_direction():
    # V = 2: KL(p||q) = p log(p/q) + (1-p) log((1-p)/(1-q)); not symmetric, so
    # swapped operands fail.
    a, c = 1.25, -0.75
    S = np.array([[a, 0.0]], np.float32)
    T = np.array([[c, 0.0]], np.float32)
    p = 1 / (1 + math.exp(-a))
    q = 1 / (1 + math.exp(-c))
    ref = p * math.log(p / q) + (1 - p) * math.log((1 - p) / (1 - q))
    rev = q * math.log(q / p) + (1 - q) * math.log((1 - q) / (1 - p))
    st = _stats(S, T, np.array([0], np.int32), np.array([0.0], np.float32))
    assert abs(st.kl[0] - ref) < 1e-14
    assert abs(st.kl[0] - rev) > 1e-2


def test_kl_uniform_teacher_is_logV_minus_entropy_and_matches_torch():
    rng = np.random.default_rng(5)
    S, T, y, b = _rand_rows(rng, 6, 400, scale=3.0)
    U = np.zeros_like(S)
    st = _stats(S, U, y, b)
    ls = torch.log_softmax(torch.from_numpy(S).double(), 1)
    ent = -(ls.exp() * ls).sum(1).numpy()
    assert np.allclose(st.kl, math.log(400) - ent, atol=1e-12)
    st = _stats(S, T, y, b)
    lt = torch.log_softmax(torch.from_numpy(T).double(), 1)
    ref = torch.nn.functional.kl_div(lt, ls, log_target=True, reduction="none").sum(1).numpy()
    assert np.allclose(st.kl, ref, atol=1e-12)
    # Pinsker (Sec. 3.3): TV <= sqrt(KL / 2)
    tv = 0.5 * (ls.exp() - lt.exp()).abs().sum(1).numpy()
    assert np.all(tv <= np.sqrt(st.kl / 2) + 1e-12)


# ------------------------------------------------------------- ratio and k3
def test_ratio_is_one_and_k3_zero_when_behaviour_equals_current():
    rng = np.random.default_rng(6)
    S, T, y, _ = _rand_rows(rng, 8, 128)
    lp = torch.log_softmax(torch.from_numpy(S), 1).numpy()[np.arange(8), y]  # fp32 on purpose
    st = _stats(S, T, y, lp.astype(np.float32))
    # b is fp32, lp_s is fp64 of the same quantity: d is at rounding level
    assert np.all(np.abs(st.d) < 1e-5)
    assert np.allclose(st.rho, 1.0, atol=1e-5)
    assert np.all(st.k3 >= 0) and np.all(st.k3 < 1e-10)
    # exactly representable case: V = 2 with equal logits gives lp = -log 2
    S2 = np.zeros((1, 2), np.float32)
    b2 = np.array([np.float32(-math.log(2))])
    st = _stats(S2, S2, np.array([1], np.int32), b2)
    assert abs(st.d[0]) < 3e-8 and st.k3[0] < 1e-15


def test_k3_expectation_under_behaviour_is_the_rollout_kl():
    # Enumerate every y on a tiny vocabulary:
    #   sum_y pi_r(y) * k3(pi_t(y)/pi_r(y)) = KL(pi_t || pi_r)   (Eq. 10, first row)
    rng = np.random.default_rng(7)
    for V in (3, 8, 21):
        cur = rng.standard_normal(V) * 1.5
        old = cur + rng.standard_normal(V) * 2.0
        lp_cur = torch.log_softmax(torch.tensor(cur), 0).numpy()
        lp_old = torch.log_softmax(torch.tensor(old), 0).numpy()
        kl_cur_old = float(np.sum(np.exp(lp_cur) * (lp_cur - lp_old)))
        kl_old_cur = float(np.sum(np.exp(lp_old) * (lp_old - lp_cur)))
        S = np.tile(cur.astype(np.float32), (V, 1))
        # behaviour log-probs must be fp32 inputs: recompute the identity on the widened values
        S64 = S.astype(np.float64)
        lp_cur32 = S64[0] - math.log(np.sum(np.exp(S64[0])))
        b = lp_old.astype(np.float32)
        pr = np.exp(b.astype(np.float64))  # not exactly normalised after rounding
        st = _stats(S, S, np.arange(V, dtype=np.int32), b)
        lhs = float(np.sum(pr * st.k3))
        # exact identity for an unnormalised reference measure pr:
        # sum pr*(rho log rho - rho + 1) = sum pt*log(pt/pr) - 1 + sum pr
        rhs = float(np.sum(np.exp(lp_cur32) * (lp_cur32 - b.astype(np.float64))) - 1.0 + pr.sum())
        assert abs(lhs - rhs) < 1e-12
        assert abs(lhs - kl_cur_old) < 1e-5 * max(1.0, kl_cur_old)   # the direction of Eq. 10
        assert abs(lhs - kl_old_cur) > 0.02 * kl_cur_old             # not the other direction


def test_k3_small_d_series_and_sign():
    S = np.zeros((3, 2), np.float32)
    base = -math.log(2)
    ds = np.array([1e-4, -1e-4, 0.5])
    b = (base - ds).astype(np.float32)
    st = _stats(S, S, np.zeros(3, np.int32), b)
    d = st.d
    series = d**2 / 2 + d**3 / 3 + d**4 / 8
    assert np.allclose(st.k3[:2], series[:2], rtol=1e-6)
    assert abs(st.k3[2] - (math.exp(d[2]) * d[2] - math.exp(d[2]) + 1)) < 1e-15
    assert np.all(st.k3 >= 0)
    assert np.allclose(st.rho, np.exp(d), rtol=1e-15)


# ------------------------------------------------------- masks and bad ids
def test_masked_and_out_of_range_rows_are_zero_and_invalid():
    rng = np.random.default_rng(8)
    S, T, y, b = _rand_rows(rng, 6, 40)
    mask = np.array([1, 0, 1, 1, 1, 1], np.uint8)
    sid = np.array([0, 0, 1, 1, 2, 5], np.int32)
    y = y.copy()
    y[2], y[3] = -1, 40
    st = orc.token_stats(S, T, y, b, mask, sid, 3)
    assert list(st.valid) == [1, 0, 0, 0, 1, 0]
    for name in ("lse_s", "lse_t", "lp_s", "lp_t", "kl", "d", "rho", "k3"):
        assert np.all(getattr(st, name)[[1, 2, 3, 5]] == 0.0)
    acc = np.zeros((3, 3))
    orc.sample_accumulate(acc, sid, st)
    assert acc[0, 0] == 1 and acc[1, 0] == 0 and acc[2, 0] == 1
    assert acc[0, 2] == st.kl[0] and acc[2, 1] == st.k3[4]


# ----------------------------------------------------------------- freshness
def test_freshness_golden_closed_forms():
    cases = json.load(open(GOLDEN))["freshness"]
    for c in cases:
        cnt = float(c["cnt"])
        acc = np.array([[cnt, c["D_roll"] * cnt, 0.7 * cnt]])
        fr = orc.sample_freshness(acc, [c["tau"]], [c["H"]], [c["D_sup"]], c["alpha"], c["beta"], c["xi"])
        assert abs(fr.f[0] - c["f"]) <= 1e-12 * max(1.0, abs(c["f"])), c
        assert abs(fr.w[0] - c["w"]) <= 1e-12, c
        assert abs(fr.m[0] - c["m"]) <= 1e-12, c


def test_freshness_hand_value_and_special_cases():
    # D_roll = 0.04, D_sup = 0.09, alpha = 1, beta = 2, tau = 3:
    # f = exp(-(0.2 + 0.6)) / 4
    acc = np.array([[10.0, 0.4, 5.0]])
    fr = orc.sample_freshness(acc, [3], [20], [0.09], 1.0, 2.0, 0.05)
    # (D_sup travels as fp32, so 0.09 is only good to ~1e-9 relative)
    assert abs(fr.f[0] - 0.25 * math.exp(-0.8)) < 1e-8
    assert abs(fr.w[0] - (0.25 * math.exp(-0.8) - 0.05)) < 1e-8
    assert fr.m[0] == 0.5 and abs(fr.ell[0] - 0.5) < 1e-15
    assert abs(fr.coef[0] - fr.w[0] / 10.0) < 1e-18
    # fresh sample: tau = 0, no drift -> f = 1
    fr = orc.sample_freshness(np.array([[4.0, 0.0, 1.0]]), [0], [4], None, 1.0, 1.0, 0.15)
    assert fr.f[0] == 1.0 and fr.w[0] == 0.85 and fr.m[0] == 1.0
    # lag-only baseline (Appendix B): alpha = beta = 0 -> 1/(tau+1)
    acc = np.array([[5.0, 2.0, 1.0]] * 4)
    fr = orc.sample_freshness(acc, [0, 1, 4, 9], [5] * 4, [0.3] * 4, 0.0, 0.0, 0.0)
    assert np.allclose(fr.f, [1.0, 0.5, 0.2, 0.1], atol=1e-15)
    # ReLU gate: f == xi -> w = 0 (excluded); f < xi -> 0
    fr = orc.sample_freshness(acc[:2], [1, 3], [5, 5], None, 0.0, 0.0, 0.5)
    assert fr.f[0] == 0.5 and fr.w[0] == 0.0 and fr.w[1] == 0.0 and np.all(fr.coef == 0)


def test_freshness_invalid_samples_and_monotonicity():
    # no aligned token / bad H / negative staleness -> f = w = m = 0, invalid (Algorithm 1)
    acc = np.array([[0.0, 0.0, 0.0], [3.0, 0.3, 0.3], [3.0, 0.3, 0.3], [3.0, 0.3, 0.3]])
    fr = orc.sample_freshness(acc, [0, 0, -1, 2], [5, 0, 5, 5], None, 1.0, 1.0, 0.1)
    assert list(fr.valid) == [0, 0, 0, 1]
    for name in ("f", "w", "m", "coef", "D_roll", "ell"):
        assert np.all(getattr(fr, name)[:3] == 0.0)
    assert fr.f[3] > 0
    # strictly decreasing in tau, D_roll and D_sup
    base = orc.sample_freshness(np.array([[2.0, 0.2, 0.0]]), [2], [2], [0.1], 1.0, 1.0, 0.0).f[0]
    assert orc.sample_freshness(np.array([[2.0, 0.2, 0.0]]), [3], [2], [0.1], 1.0, 1.0, 0.0).f[0] < base
    assert orc.sample_freshness(np.array([[2.0, 0.3, 0.0]]), [2], [2], [0.1], 1.0, 1.0, 0.0).f[0] < base
    assert orc.sample_freshness(np.array([[2.0, 0.2, 0.0]]), [2], [2], [0.2], 1.0, 1.0, 0.0).f[0] < base


# ---------------------------------------------------------------------- loss
def _tiny_batch(rng, B=3, V=11, lens=(4, 3, 5), dtype=np.float32):
    n = sum(lens)
    S, T, y, _ = _rand_rows(rng, n, V, scale=1.5)
    lp = torch.log_softmax(torch.from_numpy(S).double(), 1).numpy()[np.arange(n), y]
    b = (lp + rng.standard_normal(n) * 0.3).astype(np.float32)
    sid = np.repeat(np.arange(B, dtype=np.int32), lens)
    mask = np.ones(n, np.uint8)
    mask[1] = 0
    tau = np.array([0, 1, 2], np.int32)[:B]
    H = np.array(lens, np.int32)
    return dict(student=S, teacher=T, tokens=y, behav_logprob=b, mask=mask, sample_id=sid), tau, H


def test_loss_is_batch_mean_of_gated_sample_terms():
    rng = np.random.default_rng(9)
    chunk, tau, H = _tiny_batch(rng)
    r = orc.run_batch([chunk], 3, tau, H, None, 1.0, 1.0, 0.15, 0.1)
    fr = r.fresh
    # lambda = 0 and a wide-open gate reduce Eq. 16 to the mean of per-sample mean KLs
    r0 = orc.run_batch([chunk], 3, np.zeros(3, np.int32), H, None, 0.0, 0.0, 0.0, 0.0)
    st = r0.stats[0]
    means = [st.kl[(chunk["sample_id"] == i) & (chunk["mask"] == 1)].mean() for i in range(3)]
    assert np.all(r0.fresh.w == 1.0)
    assert abs(r0.loss - float(np.mean(means))) < 1e-14
    # linear in w, gated sample contributes nothing
    per = fr.w * (fr.ell + 0.1 * fr.D_roll)
    assert abs(r.loss - per.sum() / 3) < 1e-15
    gated = orc.run_batch([chunk], 3, np.array([0, 1, 50], np.int32), H, None, 1.0, 1.0, 0.15, 0.1)
    assert gated.fresh.w[2] == 0.0 and gated.per_sample_loss[2] == 0.0
    assert abs(gated.loss - (per[0] + per[1]) / 3) < 1e-15
    # duplicating the batch leaves the B-mean unchanged
    dup = {k: np.concatenate([v, v]) for k, v in chunk.items()}
    dup["sample_id"] = np.concatenate([chunk["sample_id"], chunk["sample_id"] + 3])
    r2 = orc.run_batch([dup], 6, np.concatenate([tau, tau]), np.concatenate([H, H]), None, 1.0, 1.0, 0.15, 0.1)
    assert abs(r2.loss - r.loss) < 1e-15


def test_chunk_split_invariance():
    rng = np.random.default_rng(10)
    chunk, tau, H = _tiny_batch(rng)
    whole = orc.run_batch([chunk], 3, tau, H, None, 1.0, 1.0, 0.15, 0.1)
    for cut in (1, 5, 6, 11):
        parts = [{k: v[:cut] for k, v in chunk.items()}, {k: v[cut:] for k, v in chunk.items()}]
        split = orc.run_batch(parts, 3, tau, H, None, 1.0, 1.0, 0.15, 0.1)
        assert np.allclose(split.acc, whole.acc, rtol=1e-15)
        assert abs(split.loss - whole.loss) < 1e-15


# ------------------------------------------------------------------ gradient
def _loss_with_frozen_w(chunk, B, w, cnt, lam):
    """Forward objective through the oracle's forward functions only, with the
    gate weights passed in as constants."""
    st = orc.token_stats(chunk["student"], chunk["teacher"], chunk["tokens"], chunk["behav_logprob"],
                         chunk["mask"], chunk["sample_id"], B)
    acc = np.zeros((B, 3))
    orc.sample_accumulate(acc, chunk["sample_id"], st)
    total = 0.0
    for i in range(B):
        if acc[i, 0] > 0:
            total += w[i] * (acc[i, 2] + lam * acc[i, 1]) / acc[i, 0]
    return total / B


def test_gradient_matches_central_finite_differences():
    rng = np.random.default_rng(11)
    chunk, tau, H = _tiny_batch(rng, V=7)
    B, lam = 3, 0.37
    r = orc.run_batch([chunk], B, tau, H, None, 1.0, 1.0, 0.05, lam)
    assert np.all(r.fresh.w > 0)
    n, V = chunk["student"].shape
    g = orc.grad_rows(chunk["student"], chunk["teacher"], chunk["tokens"], chunk["behav_logprob"],
                      chunk["mask"], chunk["sample_id"], r.fresh.coef, lam, np.arange(n))
    # fp32 storage limits the step: use h = 2^-7 (exact in fp32 for these magnitudes is not
    # guaranteed, so measure the realised step) and Richardson-free central differences.
    h = np.float32(2.0 ** -9)
    fd = np.zeros((n, V))
    for i in range(n):
        for v in range(V):
            Sp, Sm = chunk["student"].copy(), chunk["student"].copy()
            Sp[i, v] += h
            Sm[i, v] -= h
            step = float(Sp[i, v]) - float(Sm[i, v])
            lp = _loss_with_frozen_w(dict(chunk, student=Sp), B, r.fresh.w, None, lam)
            lm = _loss_with_frozen_w(dict(chunk, student=Sm), B, r.fresh.w, None, lam)
            fd[i, v] = (lp - lm) / step
    assert np.all(g[1] == 0.0) and np.all(np.abs(fd[1]) == 0.0)  # masked row
    scale = np.abs(g).max()
    assert np.max(np.abs(g - fd)) < 2e-5 * scale  # O(h^2) truncation of the central difference


def test_gradient_matches_float64_autograd_of_independent_forward():
    rng = np.random.default_rng(12)
    chunk, tau, H = _tiny_batch(rng, V=13)
    B, lam = 3, 0.2
    r = orc.run_batch([chunk], B, tau, H, None, 1.0, 1.0, 0.05, lam)
    S = torch.from_numpy(chunk["student"]).double().requires_grad_(True)
    T = torch.from_numpy(chunk["teacher"]).double()
    y = torch.from_numpy(chunk["tokens"].astype(np.int64))
    b = torch.from_numpy(chunk["behav_logprob"]).double()
    ls, lt = torch.log_softmax(S, 1), torch.log_softmax(T, 1)
    kl = torch.nn.functional.kl_div(lt, ls, log_target=True, reduction="none").sum(1)
    ratio = torch.exp(ls.gather(1, y[:, None])[:, 0] - b)
    k3 = torch.special.xlogy(ratio, ratio) - ratio + 1
    sid = torch.from_numpy(chunk["sample_id"].astype(np.int64))
    mk = torch.from_numpy(chunk["mask"]).double()
    w = torch.from_numpy(r.fresh.w)
    total = 0
    for i in range(B):
        sel = (sid == i).double() * mk
        total = total + w[i] * ((kl + lam * k3) * sel).sum() / sel.sum()
    (total / B).backward()
    assert abs(float((total / B).detach()) - r.loss) < 1e-14
    n = S.shape[0]
    g = orc.grad_rows(chunk["student"], chunk["teacher"], chunk["tokens"], chunk["behav_logprob"],
                      chunk["mask"], chunk["sample_id"], r.fresh.coef, lam, np.arange(n))
    assert np.max(np.abs(g - S.grad.numpy())) < 1e-14


def test_gradient_structure():
    rng = np.random.default_rng(13)
    chunk, tau, H = _tiny_batch(rng, V=19)
    r = orc.run_batch([chunk], 3, np.array([0, 1, 40], np.int32), H, None, 1.0, 1.0, 0.15, 0.1)
    n = chunk["student"].shape[0]
    args = (chunk["tokens"], chunk["behav_logprob"], chunk["mask"], chunk["sample_id"])
    g = orc.grad_rows(chunk["student"], chunk["teacher"], *args, r.fresh.coef, 0.1, np.arange(n))
    # both terms are tangent to the simplex: every row sums to zero
    assert np.max(np.abs(g.sum(1))) < 1e-15
    # masked row and rows of the gated sample (staleness 40) are exactly zero
    assert np.all(g[1] == 0) and np.all(g[chunk["sample_id"] == 2] == 0)
    assert np.any(g[0] != 0)
    # row subset selection returns the same rows
    sub = orc.grad_rows(chunk["student"], chunk["teacher"], *args, r.fresh.coef, 0.1, np.array([5, 0]))
    assert np.array_equal(sub[0], g[5]) and np.array_equal(sub[1], g[0])
    # teacher == student and behaviour == current policy: stationary point, gradient ~ 0
    lp = torch.log_softmax(torch.from_numpy(chunk["student"]).double(), 1).numpy()[np.arange(n), chunk["tokens"]]
    g0 = orc.grad_rows(chunk["student"], chunk["student"], chunk["tokens"], lp.astype(np.float32),
                       chunk["mask"], chunk["sample_id"], np.ones(3), 0.1, np.arange(n))
    assert np.max(np.abs(g0)) < 1e-7  # d is the fp32 rounding of b, about 1e-7
    # lambda only touches the anchor term: at lambda = 0 the gradient of row n is
    # coef * p (log p - log q - kl), which vanishes when teacher == student
    g1 = orc.grad_rows(chunk["student"], chunk["student"], *args, np.ones(3), 0.0, np.arange(n))
    assert np.max(np.abs(g1)) < 1e-15


def test_vocabulary_permutation_invariance():
    rng = np.random.default_rng(14)
    chunk, tau, H = _tiny_batch(rng, V=23)
    perm = rng.permutation(23)
    inv = np.argsort(perm)
    pc = dict(chunk, student=chunk["student"][:, perm], teacher=chunk["teacher"][:, perm],
              tokens=inv[chunk["tokens"]].astype(np.int32))
    a = orc.run_batch([chunk], 3, tau, H, None, 1.0, 1.0, 0.15, 0.1)
    p = orc.run_batch([pc], 3, tau, H, None, 1.0, 1.0, 0.15, 0.1)
    assert np.allclose(a.fresh.f, p.fresh.f, rtol=1e-13) and abs(a.loss - p.loss) < 1e-14


# ---------------------------------------------------------------- supervision drift, entropy, refresh rule
def test_row_divergence_matches_torch_float64_and_closed_forms():
    g = torch.Generator().manual_seed(11)
    A = (torch.randn(9, 37, generator=g) * 2).float()
    Bm = (A + torch.randn(9, 37, generator=g)).float()
    mask = np.array([1, 1, 0, 1, 1, 1, 0, 1, 1], np.uint8)
    kl, ent = orc.row_divergence(A, Bm, mask)
    la, lb = torch.log_softmax(A.double(), 1), torch.log_softmax(Bm.double(), 1)
    ref_kl = torch.nn.functional.kl_div(lb, la, log_target=True, reduction="none").sum(1).numpy()
    ref_ent = torch.distributions.Categorical(logits=A.double()).entropy().numpy()
    m = mask.astype(bool)
    assert np.allclose(kl[m], ref_kl[m], rtol=1e-12, atol=1e-14) and np.all(kl[~m] == 0)
    assert np.allclose(ent[m], ref_ent[m], rtol=1e-12, atol=1e-14) and np.all(ent[~m] == 0)
    assert np.all(kl[m] > 0)
    # direction: KL(first || second), not the reverse
    rev = torch.nn.functional.kl_div(la, lb, log_target=True, reduction="none").sum(1).numpy()
    assert not np.allclose(kl[m], rev[m], rtol=1e-3)
    # V = 2: Bernoulli closed forms
    a = torch.tensor([[0.3, -1.1]]); b = torch.tensor([[-0.4, 0.9]])
    p = 1 / (1 + math.exp(-(0.3 + 1.1))); q = 1 / (1 + math.exp(-(-0.4 - 0.9)))
    k2, e2 = orc.row_divergence(a, b, np.ones(1, np.uint8))
    assert abs(k2[0] - (p * math.log(p / q) + (1 - p) * math.log((1 - p) / (1 - q)))) < 1e-7
    assert abs(e2[0] - (-(p * math.log(p) + (1 - p) * math.log(1 - p)))) < 1e-7
    # identical rows: KL exactly 0; constant row: entropy log V (its maximum)
    k0, e0 = orc.row_divergence(A, A, np.ones(9, np.uint8))
    assert np.all(k0 == 0.0) and np.all(e0 <= math.log(37) + 1e-12)
    _, eu = orc.row_divergence(torch.full((1, 50), 1.5), torch.zeros(1, 50), np.ones(1, np.uint8))
    assert abs(eu[0] - math.log(50)) < 1e-12
    # a row that puts nearly all mass on one token has entropy near 0
    peaked = torch.zeros(1, 20); peaked[0, 3] = 60.0
    _, ep = orc.row_divergence(peaked, torch.zeros(1, 20), np.ones(1, np.uint8))
    assert 0 <= ep[0] < 1e-20


def test_row_divergence_is_the_token_loss_of_eq12_for_student_and_teacher():
    g = torch.Generator().manual_seed(12)
    S = torch.randn(6, 19, generator=g); T = S + 0.5 * torch.randn(6, 19, generator=g)
    st = orc.token_stats(S, T, np.zeros(6, np.int32), np.zeros(6, np.float32), np.ones(6, np.uint8),
                         np.zeros(6, np.int32), 1)
    kl, _ = orc.row_divergence(S, T, np.ones(6, np.uint8))
    assert np.allclose(kl, st.kl, rtol=1e-12, atol=1e-15)


def test_supervision_drift_means_and_empty_set():
    kl = np.array([0.1, 0.3, 0.2, 0.7]); ent = np.array([1.0, 2.0, 3.0, 4.0])
    d, m, e, cnt = orc.supervision_drift(kl, ent, [1, 0, 1, 0], [0, 0, 1, 2], [4, 2, 5], 3)
    assert np.allclose(d[:2], [0.1, 0.2]) and np.isinf(d[2]) and d[2] > 0
    assert np.allclose(m, [0.25, 0.5, 0.0]) and np.allclose(e, [1.0, 3.0, 0.0]) and np.array_equal(cnt, [1, 1, 0])
    # an empty supervision-aligned set makes the sample invalid (Algorithm 1), whatever beta is
    acc = np.array([[3.0, 0.03, 0.6]] * 3)
    for beta in (0.0, 1.0):
        fr = orc.sample_freshness(acc, [0, 1, 2], [4, 4, 4], d.astype(np.float32), 1.0, beta, 0.0)
        assert fr.valid.tolist() == [1, 1, 0] and fr.f[2] == fr.w[2] == fr.m[2] == fr.coef[2] == 0.0
        assert fr.f[0] > 0 and fr.f[1] > 0
    # and D_sup enters Eq. 11 through beta * sqrt(D_sup)
    fr = orc.sample_freshness(acc[:1], [0], [4], np.array([0.09], np.float32), 0.0, 2.0, 0.0)
    assert abs(fr.f[0] - math.exp(-2.0 * math.sqrt(np.float32(0.09)))) < 1e-12


def test_refresh_rule_operators_and_interval():
    f = [0.5, 0.25, 0.75]          # mean 0.5 exactly
    m = [0.5, 1.0, 0.75]           # mean 0.75 exactly
    ms = [0.25, 0.25, 0.25]
    means, bits, go = orc.refresh_decision(f, m, ms, 0.4, 0.7, 0.2, 500, 200)
    assert np.allclose(means, [0.5, 0.75, 0.25]) and bits == 0 and not go
    # mean f <= kappa_f triggers at equality; the alignment conditions are strict
    assert orc.refresh_decision(f, m, ms, 0.5, 0.7, 0.2, 500, 200)[1:] == (1, True)
    assert orc.refresh_decision(f, m, ms, 0.4, 0.75, 0.25, 500, 200)[1:] == (0, False)
    assert orc.refresh_decision(f, m, ms, 0.4, 0.76, 0.2, 500, 200)[1:] == (2, True)
    assert orc.refresh_decision(f, m, ms, 0.4, 0.7, 0.26, 500, 200)[1:] == (4, True)
    assert orc.refresh_decision(f, m, ms, 0.6, 0.8, 0.3, 200, 200)[1:] == (7, True)
    # at most one refresh per interval: the condition is reported but not acted on
    assert orc.refresh_decision(f, m, ms, 0.6, 0.7, 0.2, 199, 200)[1:] == (1 | 8, False)
    # one aligned set for both diagnostics: the supervision mean is the rollout mean
    means, bits, go = orc.refresh_decision(f, m, None, 0.4, 0.7, 0.76, 500, 200)
    assert means[2] == means[1] and bits == 4 and go


def test_shard_partials_hand_values_and_merge_identity():
    # one row, parts {0, ln 2} and {ln 3}: Z over the whole row is 1 + 2 + 3 = 6
    s = np.array([[0.0, math.log(2.0), math.log(3.0)]], np.float32)
    t = np.zeros_like(s)
    tok, mask = np.array([2], np.int32), np.array([1], np.uint8)
    p0 = orc.shard_partials(s[:, :2], t[:, :2], tok, mask, 0)
    p1 = orc.shard_partials(s[:, 2:], t[:, 2:], tok, mask, 2)
    l2, l3 = float(np.float32(math.log(2.0))), float(np.float32(math.log(3.0)))
    # part 0: max ln 2, Z = 1/2 + 1, A = e^{ln2 - ln2} ln 2, teacher max 0 and Z = 2, token elsewhere
    assert np.allclose(p0[0], [l2, math.exp(-l2) + 1.0, l2, 0.0, 2.0, 0.0, 0.0, 0.0], atol=1e-12)
    assert np.allclose(p1[0], [l3, 1.0, l3, 0.0, 1.0, l3, 0.0, 1.0], atol=1e-12)
    lse_s, lse_t, kl, sy, ty, found = orc.merge_partials([p0, p1])
    Z = 1.0 + math.exp(l2) + math.exp(l3)
    assert abs(lse_s[0] - math.log(Z)) < 1e-12 and abs(lse_t[0] - math.log(3.0)) < 1e-12
    # KL(p || uniform) = log 3 - H(p), p = (1, e^l2, e^l3) / Z
    p = np.array([1.0, math.exp(l2), math.exp(l3)]) / Z
    assert abs(kl[0] - (math.log(3.0) + (p * np.log(p)).sum())) < 1e-12
    assert sy[0] == l3 and ty[0] == 0.0 and found[0] == 1.0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_merged_shard_partials_equal_whole_row_statistics(dtype):
    """Any split of the vocabulary gives the whole-row normalisers, KL and log-probs."""
    rng = np.random.RandomState(7)
    n, V, B = 9, 257, 3
    S = torch.as_tensor(rng.randn(n, V) * 3).to(dtype)
    T = (S.double() + torch.as_tensor(rng.randn(n, V))).to(dtype)
    tok = rng.randint(0, V, n).astype(np.int32)
    mask = np.array([1, 1, 0, 1, 1, 1, 0, 1, 1], np.uint8)
    sid = np.repeat(np.arange(B, dtype=np.int32), 3)
    b = (rng.randn(n) - 5).astype(np.float32)
    whole = orc.token_stats(S, T, tok, b, mask, sid, B)
    for cuts in ([0, V], [0, 1, V], [0, 100, 101, 256, V], [0, 64, 128, 192, V]):
        parts = [orc.shard_partials(S[:, a:c].contiguous(), T[:, a:c].contiguous(), tok, mask, a)
                 for a, c in zip(cuts[:-1], cuts[1:])]
        lse_s, lse_t, kl, sy, ty, found = orc.merge_partials(parts)
        ok = mask.astype(bool)
        assert np.array_equal(found[ok], np.ones(ok.sum())) and np.all(found[~ok] == 0)
        assert np.allclose(lse_s[ok], whole.lse_s[ok], rtol=0, atol=1e-12)
        assert np.allclose(lse_t[ok], whole.lse_t[ok], rtol=0, atol=1e-12)
        assert np.allclose(kl[ok], whole.kl[ok], rtol=0, atol=1e-11)
        assert np.allclose((sy - lse_s)[ok], whole.lp_s[ok], rtol=0, atol=1e-12)
        assert np.allclose((ty - lse_t)[ok], whole.lp_t[ok], rtol=0, atol=1e-12)
        assert np.all(lse_s[~ok] == 0) and np.all(kl[~ok] == 0)
    # a token outside every part is reported as not found
    far = orc.shard_partials(S[:, :10].contiguous(), T[:, :10].contiguous(), np.full(n, 200, np.int32), mask, 0)
    assert np.all(orc.merge_partials([far])[5] == 0)


# ------------------------------------------------- sampled-token form of the token loss
def test_sampled_token_loss_expectation_is_the_full_vocabulary_reverse_kl():
    # Enumerate every y on a tiny vocabulary, y ~ pi_r:
    #   sum_y pi_r(y) rho(y) (log p_s(y) - log p_t(y)) = KL(p_s || p_t)        (Eq. 12)
    # with rho(y) = p_s(y) / pi_r(y); exact when pi_r is carried as the fp32 log-probs the path gets.
    rng = np.random.default_rng(31)
    for V in (2, 5, 13):
        s = (rng.standard_normal(V) * 1.5).astype(np.float32)
        t = (s + rng.standard_normal(V)).astype(np.float32)
        old = s + rng.standard_normal(V) * 0.7
        b = torch.log_softmax(torch.tensor(old, dtype=torch.float64), 0).numpy().astype(np.float32)
        S, T = np.tile(s, (V, 1)), np.tile(t, (V, 1))
        st = _stats(S, T, np.arange(V, dtype=np.int32), b)
        tl = orc.token_loss(st, orc.SAMPLED_KL)
        pr = np.exp(b.astype(np.float64))
        lhs = float(np.sum(pr * tl))
        assert abs(lhs - st.kl[0]) < 1e-12          # the oracle's own full-vocabulary token loss
        lp_s = torch.log_softmax(torch.tensor(s, dtype=torch.float64), 0)
        lp_t = torch.log_softmax(torch.tensor(t, dtype=torch.float64), 0)
        assert abs(lhs - float(torch.sum(lp_s.exp() * (lp_s - lp_t)))) < 1e-12   # and the definition
        # the other direction of the KL is a different number
        assert abs(lhs - float(torch.sum(lp_t.exp() * (lp_t - lp_s)))) > 1e-3
        # a single sampled term may be negative, the full-vocabulary loss is not
        assert tl.min() < 0 < st.kl[0]


def test_sampled_token_loss_special_cases():
    rng = np.random.default_rng(32)
    S, T, y, _ = _rand_rows(rng, 6, 9)
    lp = torch.log_softmax(torch.from_numpy(S).double(), 1).numpy()[np.arange(6), y]
    # behaviour = current and teacher = student: ratio 1, log-ratio 0, loss 0, gradient 0
    st = _stats(S, S, y, lp.astype(np.float32))
    assert np.all(orc.token_loss(st, orc.SAMPLED_KL) == 0.0)
    coef = np.array([0.25])
    g = orc.grad_rows(S, S, y, lp.astype(np.float32), np.ones(6, np.uint8), np.zeros(6, np.int32), coef, 0.3,
                      np.arange(6), loss_kind=orc.SAMPLED_KL)
    assert np.abs(g).max() < 1e-7   # d = lp_s - fp32(lp_s) is a rounding residue, not zero
    # hand value: V = 2, s = (0, ln 3), t = (0, 0), token 1, behaviour log-prob ln(1/2):
    # p_s = (1/4, 3/4), p_t = (1/2, 1/2), rho = (3/4)/(1/2) = 3/2, r = ln(3/2), loss = 1.5 ln 1.5
    s2 = np.array([[0.0, math.log(3.0)]], np.float32)
    t2 = np.zeros((1, 2), np.float32)
    st2 = _stats(s2, t2, np.array([1], np.int32), np.array([math.log(0.5)], np.float32))
    assert abs(orc.token_loss(st2, orc.SAMPLED_KL)[0] - 1.5 * math.log(1.5)) < 1e-6
    # masked rows contribute nothing
    m = np.array([1, 0, 1, 1, 0, 1], np.uint8)
    stm = _stats(S, T, y, lp.astype(np.float32), mask=m)
    tlm = orc.token_loss(stm, orc.SAMPLED_KL)
    assert np.all(tlm[m == 0] == 0.0) and np.all(tlm[m == 1] != 0.0)


def test_sampled_gradient_expectation_is_the_full_vocabulary_gradient():
    # sum_y pi_r(y) * (gradient of the sampled form with token y) = gradient of the full-vocabulary
    # form, for lambda = 0 (the anchor is the same term in both forms and is pinned separately)
    rng = np.random.default_rng(33)
    for V in (3, 7):
        s = (rng.standard_normal(V) * 1.5).astype(np.float32)
        t = (s + rng.standard_normal(V)).astype(np.float32)
        b = torch.log_softmax(torch.tensor(s + rng.standard_normal(V) * 0.5, dtype=torch.float64), 0).numpy().astype(np.float32)
        S, T = np.tile(s, (V, 1)), np.tile(t, (V, 1))
        y = np.arange(V, dtype=np.int32)
        ones, zeros = np.ones(V, np.uint8), np.zeros(V, np.int32)
        coef = np.array([1.0])
        gs = orc.grad_rows(S, T, y, b, ones, zeros, coef, 0.0, np.arange(V), loss_kind=orc.SAMPLED_KL)
        gf = orc.grad_rows(S, T, y, b, ones, zeros, coef, 0.0, np.array([0]))
        pr = np.exp(b.astype(np.float64))[:, None]
        assert np.abs((pr * gs).sum(0) - gf[0]).max() < 1e-12


def test_sampled_gradient_matches_central_finite_differences_and_structure():
    rng = np.random.default_rng(34)
    chunk, tau, H = _tiny_batch(rng, V=7)
    B, lam = 3, 0.37
    r = orc.run_batch([chunk], B, tau, H, None, 1.0, 1.0, 0.05, lam, loss_kind=orc.SAMPLED_KL)
    assert np.all(r.fresh.w > 0)
    n, V = chunk["student"].shape
    g = orc.grad_rows(chunk["student"], chunk["teacher"], chunk["tokens"], chunk["behav_logprob"],
                      chunk["mask"], chunk["sample_id"], r.fresh.coef, lam, np.arange(n), loss_kind=orc.SAMPLED_KL)
    st0 = r.stats[0]
    reward = st0.lp_s - st0.lp_t          # held constant: the importance ratio carries the derivative
    cnt = np.bincount(chunk["sample_id"][st0.valid.astype(bool)], minlength=B)

    def surrogate(S):
        st = orc.token_stats(S, chunk["teacher"], chunk["tokens"], chunk["behav_logprob"], chunk["mask"],
                             chunk["sample_id"], B)
        per_tok = st.valid * (st.rho * reward + lam * st.k3)
        tot = 0.0
        for i in range(B):
            tot += r.fresh.w[i] * per_tok[chunk["sample_id"] == i].sum() / cnt[i]
        return tot / B

    h = np.float32(2.0 ** -9)
    fd = np.zeros((n, V))
    for i in range(n):
        for v in range(V):
            Sp, Sm = chunk["student"].copy(), chunk["student"].copy()
            Sp[i, v] += h
            Sm[i, v] -= h
            fd[i, v] = (surrogate(Sp) - surrogate(Sm)) / (float(Sp[i, v]) - float(Sm[i, v]))
    assert np.all(g[1] == 0.0) and np.all(fd[1] == 0.0)   # masked row
    assert np.max(np.abs(g - fd)) < 2e-5 * np.abs(g).max()
    assert np.abs(g.sum(1)).max() < 1e-15                  # tangent to the simplex
    # the per-sample loss is the mean of the sampled token losses, the objective as in Eq. 16
    tl = orc.token_loss(orc.token_stats(chunk["student"], chunk["teacher"], chunk["tokens"], chunk["behav_logprob"],
                                        chunk["mask"], chunk["sample_id"], B), orc.SAMPLED_KL)
    ell = np.array([tl[(chunk["sample_id"] == i) & (chunk["mask"] == 1)].mean() for i in range(B)])
    assert np.allclose(r.fresh.ell, ell, rtol=1e-14)
    assert abs(r.loss - float(np.mean(r.fresh.w * (ell + lam * r.fresh.D_roll)))) < 1e-15
    # a gated sample's rows get zeros
    gated = orc.grad_rows(chunk["student"], chunk["teacher"], chunk["tokens"], chunk["behav_logprob"], chunk["mask"],
                          chunk["sample_id"], np.array([0.1, 0.0, 0.2]), lam, np.arange(n), loss_kind=orc.SAMPLED_KL)
    assert np.all(gated[chunk["sample_id"] == 1] == 0.0)
