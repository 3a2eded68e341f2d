"""ctypes front end of the fp64 CPU oracle (``fopd_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module; the CUDA library and its
binding never do, and this module imports nothing from them.

The functions mirror the C entry points one to one and add ``run_batch``, which
strings them together in the order of Algorithm 1: per-token statistics for every
chunk, per-sample sums, freshness and gate, then the objective of Eq. 16.
Logits are numpy arrays of dtype ``float32`` or ``uint16`` (bf16 bit patterns);
torch CPU tensors are accepted and reinterpreted without a copy.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fopd_oracle.c")
_LIB = os.path.join(_HERE, "libfopd_oracle.so")

BF16, F32 = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_loss.restype = ctypes.c_double
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_threads(n: int) -> None:
    lib().oracle_set_threads(ctypes.c_int(int(n)))


def _logits(a):
    """numpy view + dtype code of a logits array (torch CPU tensor or numpy)."""
    if hasattr(a, "detach"):  # torch tensor
        import torch

        a = a.detach().cpu().contiguous()
        if a.dtype == torch.bfloat16:
            a = a.view(torch.int16).numpy().view(np.uint16)
        elif a.dtype == torch.float32:
            a = a.numpy()
        else:
            raise TypeError(f"logits must be bf16 or fp32, got {a.dtype}")
    if a.dtype == np.uint16:
        return np.ascontiguousarray(a), BF16
    if a.dtype == np.float32:
        return np.ascontiguousarray(a), F32
    raise TypeError(f"logits must be uint16 (bf16 bits) or float32, got {a.dtype}")


def _np(a, dtype):
    if hasattr(a, "detach"):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, dtype=dtype)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class TokenStats:
    lse_s: np.ndarray
    lse_t: np.ndarray
    lp_s: np.ndarray
    lp_t: np.ndarray
    kl: np.ndarray
    d: np.ndarray
    rho: np.ndarray
    k3: np.ndarray
    valid: np.ndarray


def token_stats(student, teacher, tokens, behav_logprob, mask, sample_id, B) -> TokenStats:
    """Per-token quantities of one chunk (softmax normalisers, gathered
    log-probs, reverse-KL token loss of Eq. 12, ratio and drift integrand of
    Eq. 10)."""
    S, dt = _logits(student)
    T, dt2 = _logits(teacher)
    assert dt == dt2 and S.shape == T.shape and S.ndim == 2
    n, V = S.shape
    y = _np(tokens, np.int32)
    b = _np(behav_logprob, np.float32)
    mk = _np(mask, np.uint8)
    sid = _np(sample_id, np.int32)
    outs = [np.zeros(n, dtype=np.float64) for _ in range(8)]
    valid = np.zeros(n, dtype=np.uint8)
    lib().oracle_token_stats(
        _p(S), _p(T), ctypes.c_int(dt), ctypes.c_int64(n), ctypes.c_int64(V), ctypes.c_int64(V),
        _p(y), _p(b), _p(mk), _p(sid), ctypes.c_int32(B), *[_p(o) for o in outs], _p(valid),
    )
    return TokenStats(*outs, valid)


def sample_accumulate(acc, sample_id, stats: TokenStats) -> None:
    """acc[B,3] += {count, sum k3, sum kl} over the aligned rows of a chunk."""
    sid = _np(sample_id, np.int32)
    assert acc.dtype == np.float64 and acc.flags.c_contiguous and acc.shape[1] == 3
    lib().oracle_sample_accumulate(
        ctypes.c_int64(len(sid)), ctypes.c_int32(acc.shape[0]), _p(sid), _p(stats.valid),
        _p(stats.kl), _p(stats.k3), _p(acc),
    )


@dataclass
class Freshness:
    f: np.ndarray
    w: np.ndarray
    D_roll: np.ndarray
    ell: np.ndarray
    m: np.ndarray
    coef: np.ndarray
    valid: np.ndarray


def sample_freshness(acc, tau, H, d_sup, alpha, beta, xi) -> Freshness:
    """Eq. 11 freshness, Eq. 13 ReLU gate, alignment ratio and token weight."""
    B = acc.shape[0]
    tau = _np(tau, np.int32)
    H = _np(H, np.int32)
    ds = None if d_sup is None else _np(d_sup, np.float32)
    outs = [np.zeros(B, dtype=np.float64) for _ in range(6)]
    valid = np.zeros(B, dtype=np.uint8)
    lib().oracle_sample_freshness(
        ctypes.c_int32(B), _p(np.ascontiguousarray(acc)), _p(tau), _p(H),
        _p(ds) if ds is not None else None,
        ctypes.c_double(alpha), ctypes.c_double(beta), ctypes.c_double(xi),
        *[_p(o) for o in outs], _p(valid),
    )
    return Freshness(*outs, valid)


def loss(fr: Freshness, lam):
    """Eq. 16 / Algorithm 1: (1/B) sum_i w_i (l_i + lambda D_roll_i)."""
    per = np.zeros(len(fr.w), dtype=np.float64)
    total = lib().oracle_loss(
        ctypes.c_int32(len(fr.w)), _p(fr.w), _p(fr.ell), _p(fr.D_roll), ctypes.c_double(lam), _p(per)
    )
    return float(total), per


FULL_KL, SAMPLED_KL = 0, 1  # forms of the token loss of Eq. 12


def token_loss(st: TokenStats, loss_kind: int = FULL_KL) -> np.ndarray:
    """Per-token loss of a chunk: the full-vocabulary reverse KL (loss_kind 0) or its
    sampled-token form rho_n (lp_s - lp_t) on the stored token (loss_kind 1)."""
    if loss_kind == FULL_KL:
        return st.kl
    out = np.zeros_like(st.kl)
    lib().oracle_sampled_token_loss(ctypes.c_int64(len(out)), _p(st.lp_s), _p(st.lp_t), _p(st.rho),
                                    _p(st.valid), _p(out))
    return out


def grad_rows(student, teacher, tokens, behav_logprob, mask, sample_id, coef, lam, rows, loss_kind: int = FULL_KL):
    """d L / d student logits for the listed rows, [len(rows), V] float64."""
    S, dt = _logits(student)
    T, dt2 = _logits(teacher)
    assert dt == dt2 and S.shape == T.shape
    n, V = S.shape
    y = _np(tokens, np.int32)
    b = _np(behav_logprob, np.float32)
    mk = _np(mask, np.uint8)
    sid = _np(sample_id, np.int32)
    coef = _np(coef, np.float64)
    rows = _np(rows, np.int64)
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < n)
    out = np.zeros((len(rows), V), dtype=np.float64)
    fn = lib().oracle_grad_rows if loss_kind == FULL_KL else lib().oracle_grad_rows_sampled
    fn(
        _p(S), _p(T), ctypes.c_int(dt), ctypes.c_int64(V), ctypes.c_int64(V), _p(y), _p(b), _p(mk),
        _p(sid), ctypes.c_int32(len(coef)), _p(coef), ctypes.c_double(lam), _p(rows),
        ctypes.c_int64(len(rows)), _p(out),
    )
    return out


def row_divergence(first, second, mask):
    """Row-wise KL(softmax(first) || softmax(second)) and entropy of softmax(first)
    at rows with mask = 1 (Eq. 10 second row when the two are the teacher under
    the current and the stored context)."""
    A, dt = _logits(first)
    Bm, dt2 = _logits(second)
    assert dt == dt2 and A.shape == Bm.shape
    n, V = A.shape
    mk = _np(mask, np.uint8)
    kl, ent = np.zeros(n), np.zeros(n)
    lib().oracle_row_divergence(_p(A), _p(Bm), ctypes.c_int(dt), ctypes.c_int64(n), ctypes.c_int64(V),
                                ctypes.c_int64(V), _p(mk), _p(kl), _p(ent))
    return kl, ent


def supervision_drift(kl, entropy, mask, sample_id, H, B):
    """D_sup_i = mean of the row KLs over U_i^sup (Eq. 10), m_sup_i = |U_i^sup| / H_i
    (Algorithm 1), mean entropy; an empty U_i^sup gives D_sup = +inf, m_sup = 0."""
    sid = np.asarray(sample_id)
    m = np.asarray(mask).astype(bool)
    H = np.asarray(H, dtype=np.float64)
    cnt = np.zeros(B)
    skl = np.zeros(B)
    sen = np.zeros(B)
    for n in range(len(sid)):  # plain loop: the definition
        if m[n]:
            cnt[sid[n]] += 1.0
            skl[sid[n]] += kl[n]
            sen[sid[n]] += entropy[n]
    d_sup = np.where(cnt > 0, skl / np.maximum(cnt, 1.0), np.inf)
    m_sup = np.where((cnt > 0) & (H > 0), cnt / np.where(H > 0, H, 1.0), 0.0)
    ment = np.where(cnt > 0, sen / np.maximum(cnt, 1.0), 0.0)
    return d_sup, m_sup, ment, cnt


def refresh_decision(f, m_roll, m_sup, kappa_f, kappa_roll, kappa_sup, steps_since_refresh, min_interval):
    """Eq. 14 buffer means and the Eq. 15 rule (mean f <= kappa_f or mean m < kappa),
    at most one refresh per min_interval steps (Appendix B).  Returns (means, bits, refresh)."""
    f = np.asarray(f, dtype=np.float64)
    mr = np.asarray(m_roll, dtype=np.float64)
    ms = mr if m_sup is None else np.asarray(m_sup, dtype=np.float64)
    means = np.array([f.mean(), mr.mean(), ms.mean()])
    bits = (1 if means[0] <= kappa_f else 0) | (2 if means[1] < kappa_roll else 0) | (4 if means[2] < kappa_sup else 0)
    due = steps_since_refresh >= min_interval
    refresh = bool(bits) and due
    if bits and not due:
        bits |= 8
    return means, bits, refresh


def _to_f64(a):
    """Logits (bf16 bit patterns, fp32, or a torch CPU tensor of either) as float64."""
    x, dt = _logits(a)
    if dt == BF16:
        return (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return x.astype(np.float64)


def shard_partials(student_shard, teacher_shard, tokens, mask, v0):
    """Partial sums of the columns [v0, v0 + W) of every row, for logits whose vocabulary
    is split over several holders (Sec. 4.1's softmax normaliser and Eq. 12's sum, taken
    over a part of the vocabulary): columns m_s = max s, Z_s = sum e^{s - m_s},
    A_s = sum e^{s - m_s} (s - t), m_t, Z_t, then the stored token's two logits and a
    flag when the token lies in this part (zeros otherwise).  Rows with mask = 0: zeros."""
    S, T = _to_f64(student_shard), _to_f64(teacher_shard)
    n, W = S.shape
    y = _np(tokens, np.int64) - int(v0)
    mk = _np(mask, np.uint8).astype(bool)
    out = np.zeros((n, 8), dtype=np.float64)
    for r in range(n):
        if not mk[r]:
            continue
        ms, mt = S[r].max(), T[r].max()
        es = np.exp(S[r] - ms)
        out[r, :5] = ms, es.sum(), (es * (S[r] - T[r])).sum(), mt, np.exp(T[r] - mt).sum()
        if 0 <= y[r] < W:
            out[r, 5:] = S[r, y[r]], T[r, y[r]], 1.0
    return out


def merge_partials(parts):
    """Whole-row normalisers, KL and stored-token logits from the partial sums of all parts
    ([n_parts, n_rows, 8]): lse = log sum_k Z_k e^{m_k}, sum_v p_s(v)(s_v - t_v) =
    sum_k A_k e^{m_k} / sum_k Z_k e^{m_k}.  Returns (lse_s, lse_t, kl, s_y, t_y, found)."""
    P = np.asarray(parts, dtype=np.float64)
    live = P[:, :, 1] > 0  # parts of rows with mask = 1
    Ms = np.where(live, P[:, :, 0], -np.inf).max(0)
    Mt = np.where(live, P[:, :, 3], -np.inf).max(0)
    ok = live.any(0)
    Ms, Mt = np.where(ok, Ms, 0.0), np.where(ok, Mt, 0.0)
    ws = np.where(live, np.exp(P[:, :, 0] - Ms), 0.0)
    wt = np.where(live, np.exp(P[:, :, 3] - Mt), 0.0)
    Zs, As, Zt = (ws * P[:, :, 1]).sum(0), (ws * P[:, :, 2]).sum(0), (wt * P[:, :, 4]).sum(0)
    with np.errstate(divide="ignore", invalid="ignore"):
        lse_s, lse_t = Ms + np.log(Zs), Mt + np.log(Zt)
        kl = As / Zs - lse_s + lse_t
    found = P[:, :, 7].sum(0)
    sy, ty = (P[:, :, 5] * P[:, :, 7]).sum(0), (P[:, :, 6] * P[:, :, 7]).sum(0)
    z = lambda a: np.where(ok, a, 0.0)
    return z(lse_s), z(lse_t), z(kl), sy, ty, found


@dataclass
class BatchResult:
    stats: list  # TokenStats per chunk
    acc: np.ndarray  # [B,3]
    fresh: Freshness
    loss: float
    per_sample_loss: np.ndarray


def run_batch(chunks, B, tau, H, d_sup, alpha, beta, xi, lam, loss_kind: int = FULL_KL) -> BatchResult:
    """Algorithm 1's measurement phase then its minibatch objective, over a
    batch supplied as a list of chunks.  Each chunk is a dict with keys
    student, teacher, tokens, behav_logprob, mask, sample_id."""
    acc = np.zeros((B, 3), dtype=np.float64)
    stats = []
    for c in chunks:
        st = token_stats(c["student"], c["teacher"], c["tokens"], c["behav_logprob"],
                         c["mask"], c["sample_id"], B)
        if loss_kind != FULL_KL:  # the per-sample mean of Eq. 12 is taken over this form of the token loss
            st.kl = token_loss(st, loss_kind)
        sample_accumulate(acc, c["sample_id"], st)
        stats.append(st)
    fr = sample_freshness(acc, tau, H, d_sup, alpha, beta, xi)
    total, per = loss(fr, lam)
    return BatchResult(stats, acc, fr, total, per)
