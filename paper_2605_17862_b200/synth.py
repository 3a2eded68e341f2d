"""Seeded synthetic inputs shaped like the paper's three workloads.

This module only *generates inputs*: batch structure (ragged lengths, loss
masks, sample ids, staleness) with numpy, and logits / sampled tokens /
behaviour log-probs with torch on whatever device is asked for.  It holds none
of the method's arithmetic and is the one module both the CUDA tests and the
CPU oracle tests draw inputs from; the same generated bits go to both sides.

The five workloads follow the benchmark configurations (reasoning, tool-use and
coding-agent shapes of the paper's Sec. 5 / Appendix B task families, a tiny
fp32 correctness case and a roofline sweep); the paper's datasets and model
outputs are not reproduced, only their shapes.  ``scale`` shrinks rows and
vocabulary for tests that must run on the CPU oracle in seconds.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch


@dataclass
class Workload:
    name: str
    B: int
    V: int
    dtype: torch.dtype
    chunk_rows: int
    sample_id: np.ndarray  # [N] int32, non-decreasing
    mask: np.ndarray  # [N] uint8
    tau: np.ndarray  # [B] int32 staleness in policy versions
    H: np.ndarray  # [B] int32 response length (padding excluded, masked tool output included)
    sigma_s: float = 3.0
    boost_frac: float = 0.01
    boost: float = 8.0
    sigma_t: float = 1.0
    sigma_b: float = 0.3
    seed: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def n_rows(self) -> int:
        return int(self.sample_id.shape[0])

    @property
    def n_chunks(self) -> int:
        return (self.n_rows + self.chunk_rows - 1) // self.chunk_rows

    def chunk_range(self, j: int):
        lo = j * self.chunk_rows
        return lo, min(lo + self.chunk_rows, self.n_rows)


# Hyper-parameters used by every test and benchmark line.  The paper never
# prints values for alpha, beta, xi, lambda (they are tuned on a pilot split),
# so these are this repository's choice: with xi = 0.15 a sample with
# staleness >= 6 is always gated out and staleness 4-5 sits near the gate.
def f32_params(alpha=1.0, beta=1.0, xi=0.15, lam=0.1) -> dict:
    """Hyper-parameters rounded to fp32 once, as Python floats.  The C ABI carries
    them as ``float``; a checker that is to see identical inputs must be handed
    these rounded values, not the decimal literals (0.15 is not an fp32 number)."""
    return {k: float(np.float32(v)) for k, v in dict(alpha=alpha, beta=beta, xi=xi, lam=lam).items()}


DEFAULT_PARAMS = f32_params()


def _scaled_vocab(full: int, scale: float) -> int:
    """Scaled vocabulary, kept a multiple of 8 so that bf16 rows stay 16-byte aligned."""
    return max(96, (int(full * scale) + 7) // 8 * 8)


def _packed(lengths):
    sid = np.repeat(np.arange(len(lengths), dtype=np.int32), lengths)
    return sid


def tiny(scale: float = 1.0) -> Workload:
    """Config 1: 4 x 256 tokens, V = 32,000, fp32, mask all ones, staleness 0..3."""
    rng = np.random.RandomState(0)
    B, T = 4, max(8, int(256 * scale))
    V = _scaled_vocab(32000, scale)
    lengths = np.full(B, T, dtype=np.int64)
    sid = _packed(lengths)
    return Workload("tiny", B, V, torch.float32, sid.shape[0], sid, np.ones_like(sid, dtype=np.uint8),
                    rng.randint(0, 4, size=B).astype(np.int32), lengths.astype(np.int32),
                    sigma_s=2.0, boost_frac=0.0, sigma_t=0.5, sigma_b=0.2, seed=0)


def reasoning(scale: float = 1.0, V: int | None = None) -> Workload:
    """Config 2: 16 sequences padded to 2,048 rows each, lengths U[512, 2048],
    padding masked, V = 151,936, bf16, staleness 0..2."""
    rng = np.random.RandomState(1)
    B, T = 16, max(16, int(2048 * scale))
    V = V or _scaled_vocab(151936, scale)
    lengths = rng.randint(max(1, T // 4), T + 1, size=B)
    sid = np.repeat(np.arange(B, dtype=np.int32), T)
    pos = np.tile(np.arange(T), B)
    mask = (pos < np.repeat(lengths, T)).astype(np.uint8)
    return Workload("reasoning", B, V, torch.bfloat16, B * T, sid, mask,
                    rng.randint(0, 3, size=B).astype(np.int32), lengths.astype(np.int32), seed=1)


def tool_use(scale: float = 1.0, V: int | None = None) -> Workload:
    """Config 3: 32 packed sequences, lengths U[1024, 8192]; 3-10 masked
    tool-output spans of length U[50, 400] per sequence (about 30% masked);
    staleness 0..4; streamed in 16,384-row chunks that cut across samples."""
    rng = np.random.RandomState(2)
    B = 32
    V = V or _scaled_vocab(151936, scale)
    lo, hi = max(4, int(1024 * scale)), max(8, int(8192 * scale))
    lengths = rng.randint(lo, hi + 1, size=B)
    sid = _packed(lengths)
    mask = np.ones(sid.shape[0], dtype=np.uint8)
    start = 0
    for L in lengths:
        for _ in range(rng.randint(3, 11)):
            sl = max(1, int(rng.randint(50, 401) * scale))
            sl = min(sl, L)
            s0 = rng.randint(0, L - sl + 1)
            mask[start + s0:start + s0 + sl] = 0
        start += L
    return Workload("tool_use", B, V, torch.bfloat16, max(8, int(16384 * scale)), sid, mask,
                    rng.randint(0, 5, size=B).astype(np.int32), lengths.astype(np.int32), seed=2)


def coding_agent(scale: float = 1.0, V: int | None = None) -> Workload:
    """Config 4: 8 packed sequences of 16,384-32,768 tokens, alternating
    kept / masked spans of length U[100, 2000] (about half masked), staleness
    0..8 with at least one sample at staleness >= 6, teacher noise sigma 2,
    16,384-row chunks."""
    rng = np.random.RandomState(3)
    B = 8
    V = V or _scaled_vocab(151936, scale)
    lo, hi = max(8, int(16384 * scale)), max(16, int(32768 * scale))
    lengths = rng.randint(lo, hi + 1, size=B)
    sid = _packed(lengths)
    mask = np.ones(sid.shape[0], dtype=np.uint8)
    start = 0
    for L in lengths:
        pos, keep = 0, bool(rng.randint(0, 2))
        while pos < L:
            sl = max(1, int(rng.randint(100, 2001) * scale))
            if not keep:
                mask[start + pos:start + min(L, pos + sl)] = 0
            pos += sl
            keep = not keep
        start += L
    tau = rng.randint(0, 9, size=B).astype(np.int32)
    if tau.max() < 6:
        tau[int(rng.randint(0, B))] = 6 + int(rng.randint(0, 3))
    assert tau.max() >= 6
    return Workload("coding_agent", B, V, torch.bfloat16, max(8, int(16384 * scale)), sid, mask,
                    tau, lengths.astype(np.int32), sigma_t=2.0, seed=3)


def roofline_point(n_rows: int, V: int, rows_per_sample: int = 2048) -> Workload:
    """Config 5: one point of the rows x vocabulary sweep; bf16, all tokens
    unmasked, samples of 2,048 rows, staleness 0..4."""
    rng = np.random.RandomState(4)
    rows_per_sample = min(rows_per_sample, n_rows)
    B = max(1, n_rows // rows_per_sample)
    lengths = np.full(B, rows_per_sample, dtype=np.int64)
    lengths[-1] += n_rows - B * rows_per_sample
    sid = _packed(lengths)
    return Workload(f"roofline_{n_rows}x{V}", B, V, torch.bfloat16, n_rows, sid,
                    np.ones(n_rows, dtype=np.uint8), rng.randint(0, 5, size=B).astype(np.int32),
                    lengths.astype(np.int32), seed=4)


WORKLOADS = {"tiny": tiny, "reasoning": reasoning, "tool_use": tool_use, "coding_agent": coding_agent}


def gen_rows(n_rows: int, V: int, dtype: torch.dtype, *, sigma_s: float, boost_frac: float,
             boost: float, sigma_t: float, sigma_b: float, seed: int, device="cpu",
             row_block: int = 512, row_stride: int | None = None):
    """Student / teacher logits, sampled tokens and behaviour log-probs.

    student  = round_dtype( sigma_s * N(0,1)  [+ boost on a boost_frac share of entries] )
    teacher  = round_dtype( unrounded student + sigma_t * N(0,1) )
    behaviour logits = student (as stored) + sigma_b * N(0,1), never stored
    token    ~ softmax(behaviour logits) at temperature 1 (Gumbel-max)
    behav_logprob = log_softmax(behaviour logits)[token]  (fp32, library routine)

    Generated in row blocks so a full-size chunk never needs more than a few
    fp32 temporaries of ``row_block`` rows.  Returns (student, teacher, tokens,
    behav_logprob); logits are [n_rows, row_stride] with the first V columns used.
    """
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    stride = row_stride or V
    S = torch.zeros((n_rows, stride), dtype=dtype, device=dev)
    T = torch.zeros((n_rows, stride), dtype=dtype, device=dev)
    y = torch.empty(n_rows, dtype=torch.int32, device=dev)
    b = torch.empty(n_rows, dtype=torch.float32, device=dev)
    for r0 in range(0, n_rows, row_block):
        r1 = min(n_rows, r0 + row_block)
        shape = (r1 - r0, V)
        s32 = torch.randn(shape, generator=g, device=dev) * sigma_s
        if boost_frac > 0:
            s32 += (torch.rand(shape, generator=g, device=dev) < boost_frac) * boost
        S[r0:r1, :V] = s32.to(dtype)
        s32 += torch.randn(shape, generator=g, device=dev) * sigma_t
        T[r0:r1, :V] = s32.to(dtype)
        del s32
        bh = S[r0:r1, :V].float() + torch.randn(shape, generator=g, device=dev) * sigma_b
        u = torch.rand(shape, generator=g, device=dev).clamp_(1e-20, 1.0)
        tok = torch.argmax(bh - torch.log(-torch.log(u)), dim=1)
        del u
        logp = torch.log_softmax(bh, dim=1)
        y[r0:r1] = tok.to(torch.int32)
        b[r0:r1] = logp.gather(1, tok[:, None])[:, 0]
    return S, T, y, b


def gen_chunk(wl: Workload, j: int, device="cpu", row_block: int = 512, row_stride: int | None = None):
    """All per-row inputs of chunk j of a workload, as a dict of torch tensors
    on ``device``.  Chunk j is seeded with seed * 1000 + j, so chunks can be
    regenerated independently and in any order."""
    lo, hi = wl.chunk_range(j)
    S, T, y, b = gen_rows(hi - lo, wl.V, wl.dtype, sigma_s=wl.sigma_s, boost_frac=wl.boost_frac,
                          boost=wl.boost, sigma_t=wl.sigma_t, sigma_b=wl.sigma_b,
                          seed=wl.seed * 1000 + j, device=device, row_block=row_block,
                          row_stride=row_stride)
    dev = torch.device(device)
    return dict(
        student=S, teacher=T, tokens=y, behav_logprob=b,
        mask=torch.from_numpy(wl.mask[lo:hi].copy()).to(dev),
        sample_id=torch.from_numpy(wl.sample_id[lo:hi].copy()).to(dev),
    )
