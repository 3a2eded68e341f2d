"""Calling sequence of the library for one batch, in the order of Algorithm 1:
statistics for every chunk, freshness, then the fused loss forward + backward
for every chunk and the final reduction.  Allocates the caller-owned buffers
with torch and calls the binding; no arithmetic happens here.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

from . import binding as fb


@dataclass
class BatchBuffers:
    """Caller-owned per-sample buffers of one batch of B samples."""
    B: int
    device: torch.device
    acc: torch.Tensor = None
    loss_acc: torch.Tensor = None
    status: torch.Tensor = None
    f: torch.Tensor = None
    w: torch.Tensor = None
    d_roll: torch.Tensor = None
    l_distill: torch.Tensor = None
    m_align: torch.Tensor = None
    coef: torch.Tensor = None
    buffer_means: torch.Tensor = None
    per_sample_loss: torch.Tensor = None
    loss: torch.Tensor = None

    def __post_init__(self):
        dev, B = self.device, self.B
        self.acc = torch.zeros((B, 4), dtype=torch.float64, device=dev)
        self.loss_acc = torch.zeros((B, 2), dtype=torch.float64, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        for name in ("f", "w", "d_roll", "l_distill", "m_align", "coef", "per_sample_loss"):
            setattr(self, name, torch.zeros(B, dtype=torch.float32, device=dev))
        self.buffer_means = torch.zeros(2, dtype=torch.float32, device=dev)
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)

    def reset(self):
        self.acc.zero_()
        self.loss_acc.zero_()
        self.status.zero_()


@dataclass
class RowOutputs:
    lp_s: torch.Tensor
    lp_t: torch.Tensor
    kl: torch.Tensor
    ratio: torch.Tensor
    row_ws: torch.Tensor

    @staticmethod
    def alloc(n: int, device) -> "RowOutputs":
        z = lambda: torch.empty(n, dtype=torch.float32, device=device)
        return RowOutputs(z(), z(), z(), z(), torch.empty((n, 4), dtype=torch.float32, device=device))


def measure(chunks, buf: BatchBuffers, rows=None, *, keep_row_ws=True, stream=None):
    """Measurement phase: fopd_token_stats on every chunk.  ``rows`` is an
    optional list of RowOutputs (one per chunk) receiving per-token outputs."""
    for j, ch in enumerate(chunks):
        r = rows[j] if rows is not None else None
        fb.fopd_token_stats(
            ch, buf.B, buf.acc,
            lp_s=r.lp_s if r else None, lp_t=r.lp_t if r else None, kl=r.kl if r else None,
            ratio=r.ratio if r else None, row_ws=(r.row_ws if (r and keep_row_ws) else None),
            status=buf.status, stream=stream)


def measure_student(chunks, buf: BatchBuffers, rows=None, *, stream=None):
    """Measurement phase from the student rows alone (fopd_token_stats_student): all that the
    freshness score needs.  The chunks' teacher rows are not read (and may be absent)."""
    for j, ch in enumerate(chunks):
        r = rows[j] if rows is not None else None
        student_view = fb.Chunk(ch.student, None, ch.behav_logprob, ch.tokens, ch.mask, ch.sample_id, ch.vocab,
                                ch.loss_kind)
        fb.fopd_token_stats_student(student_view, buf.B, buf.acc, lp_s=r.lp_s if r else None,
                                    ratio=r.ratio if r else None, status=buf.status, stream=stream)


def freshness(buf: BatchBuffers, tau, H, d_sup, p, stream=None):
    fb.fopd_sample_freshness(buf.acc, tau, H, d_sup, buf.B, p, coef=buf.coef, f=buf.f, w=buf.w,
                             d_roll=buf.d_roll, l_distill=buf.l_distill, m_align=buf.m_align,
                             buffer_means=buf.buffer_means, status=buf.status, stream=stream)


def optimise(chunks, dlogits, buf: BatchBuffers, p, rows=None, *, use_row_ws=True, stream=None):
    """Optimisation phase: fopd_loss_fwd_bwd on every chunk (dlogits[j] receives
    chunk j's gradient), then fopd_loss_finalize."""
    for j, ch in enumerate(chunks):
        ws = rows[j].row_ws if (rows is not None and use_row_ws) else None
        fb.fopd_loss_fwd_bwd(ch, buf.B, buf.coef, p, dlogits[j], buf.loss_acc, row_ws=ws,
                             status=buf.status, stream=stream)
    fb.fopd_loss_finalize(buf.loss_acc, buf.acc, buf.w, buf.B, p, buf.loss,
                          per_sample_loss=buf.per_sample_loss, stream=stream)


def step(chunks, dlogits, buf: BatchBuffers, tau, H, d_sup, p, rows=None, *, use_row_ws=True, stream=None):
    """One pass of the whole hot path over one batch."""
    buf.reset()
    measure(chunks, buf, rows, keep_row_ws=use_row_ws, stream=stream)
    freshness(buf, tau, H, d_sup, p, stream=stream)
    optimise(chunks, dlogits, buf, p, rows, use_row_ws=use_row_ws, stream=stream)


def step_student_stats(chunks, dlogits, buf: BatchBuffers, tau, H, d_sup, p, rows=None, *, stream=None):
    """The whole hot path with the fewest bytes: the student's statistics (V e per token), the
    freshness, then the loss forward + backward without cached statistics (3 V e per
    differentiated token)."""
    buf.reset()
    measure_student(chunks, buf, rows, stream=stream)
    freshness(buf, tau, H, d_sup, p, stream=stream)
    optimise(chunks, dlogits, buf, p, None, use_row_ws=False, stream=stream)


def to_chunk(d: dict, vocab=None, loss_kind: int = fb.LOSS_FULL_KL) -> fb.Chunk:
    return fb.Chunk(d["student"], d["teacher"], d["behav_logprob"], d["tokens"], d["mask"], d["sample_id"], vocab,
                    loss_kind)


# ---- vocabulary-sharded rows: every holder (rank) has a column range of every row ----

def gather_parts(partial: torch.Tensor, group=None) -> torch.Tensor:
    """Every holder's partial sums on every holder: [world, n_rows, 8], part k from rank k.
    The only exchange of the sharded path (32 bytes per row and holder); one process: a copy."""
    import torch.distributed as dist

    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    out = torch.empty((world,) + tuple(partial.shape), dtype=partial.dtype, device=partial.device)
    if world == 1:
        out[0].copy_(partial)
    else:
        dist.all_gather(list(out.unbind(0)), partial.contiguous(), group=group)
    return out


def step_vocab_sharded(shards, vocab_offset: int, vocab_total: int, dlogits, buf: BatchBuffers, tau, H, d_sup, p,
                       rows, *, gather=gather_parts, stream=None):
    """One pass of the whole path on a holder of the columns [vocab_offset, vocab_offset + W):
    ``shards`` are this holder's chunks (logits = its columns, tokens = full-vocabulary ids),
    ``rows`` one RowOutputs per chunk (row_ws is required), ``gather`` brings all holders'
    partial sums together (default: all-gather over the default process group)."""
    buf.reset()
    for j, sh in enumerate(shards):
        n = sh.tokens.numel()
        part = torch.empty((n, 8), dtype=torch.float32, device=buf.device)
        fb.fopd_shard_stats(sh, vocab_offset, vocab_total, part, stream=stream)
        parts = gather(part)
        r = rows[j]
        fb.fopd_shard_merge(parts, sh.behav_logprob, sh.tokens, sh.mask, sh.sample_id, vocab_total, buf.B, buf.acc,
                            r.row_ws, lp_s=r.lp_s, lp_t=r.lp_t, kl=r.kl, ratio=r.ratio, status=buf.status,
                            stream=stream)
    freshness(buf, tau, H, d_sup, p, stream=stream)
    for j, sh in enumerate(shards):
        fb.fopd_shard_loss_fwd_bwd(sh, vocab_offset, vocab_total, buf.B, buf.coef, rows[j].row_ws, p, dlogits[j],
                                   loss_acc=buf.loss_acc, stream=stream)
    fb.fopd_loss_finalize(buf.loss_acc, buf.acc, buf.w, buf.B, p, buf.loss,
                          per_sample_loss=buf.per_sample_loss, stream=stream)
