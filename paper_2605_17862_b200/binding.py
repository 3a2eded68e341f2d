"""Thin ctypes binding of libfopd.so: same names as the C ABI, torch tensors in,
pointers out.  Argument marshalling only -- every step of the path runs in the
library's CUDA kernels.  There is no CPU fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfopd.so")

FOPD_BF16, FOPD_F32 = 0, 1
LOSS_FULL_KL, LOSS_SAMPLED_KL = 0, 1  # forms of the token loss (fopd_loss_kind)

EXPORTS = (
    "fopd_token_stats", "fopd_sample_freshness", "fopd_loss_fwd_bwd", "fopd_loss_finalize",
    "fopd_check_status", "fopd_strerror", "fopd_version", "fopd_step_host", "fopd_step_host_workspace_bytes",
    "fopd_token_stats_static", "fopd_loss_fwd_bwd_plan", "fopd_row_divergence", "fopd_supervision_drift",
    "fopd_refresh_decision", "fopd_shard_stats", "fopd_shard_merge", "fopd_shard_loss_fwd_bwd",
    "fopd_loss_fwd_bwd_set_plan", "fopd_release_device_memory", "fopd_selftest_bounded_wait",
    "fopd_token_stats_student",
)


class FopdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} (status {code})")


class fopd_params(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_float), ("beta", ctypes.c_float), ("xi", ctypes.c_float),
                ("lam", ctypes.c_float)]


class fopd_chunk(ctypes.Structure):
    _fields_ = [
        ("student", ctypes.c_void_p), ("teacher", ctypes.c_void_p), ("behav_logprob", ctypes.c_void_p),
        ("tokens", ctypes.c_void_p), ("mask", ctypes.c_void_p), ("sample_id", ctypes.c_void_p),
        ("n_rows", ctypes.c_int64), ("vocab", ctypes.c_int64), ("row_stride", ctypes.c_int64),
        ("dtype", ctypes.c_int32), ("loss_kind", ctypes.c_int32),
    ]


class fopd_host_outputs(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("f", "w", "d_roll", "l_distill", "m_align", "per_sample_loss", "buffer_means", "loss",
                 "status_bits", "copied_bytes")]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libfopd.so (built in-tree by ``build.build_lib``); fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2605_17862_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32 = ctypes.c_void_p, ctypes.c_int32
        L.fopd_version.restype = ctypes.c_int
        L.fopd_strerror.restype = ctypes.c_char_p
        L.fopd_strerror.argtypes = [ctypes.c_int]
        L.fopd_token_stats.argtypes = [ctypes.POINTER(fopd_chunk), i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.fopd_token_stats_student.argtypes = [ctypes.POINTER(fopd_chunk), i32, vp, vp, vp, vp, vp]
        L.fopd_token_stats_static.argtypes = [ctypes.POINTER(fopd_chunk), i32, vp, vp, vp, vp, vp, vp, vp]
        L.fopd_sample_freshness.argtypes = [vp, vp, vp, vp, i32, fopd_params, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.fopd_loss_fwd_bwd.argtypes = [ctypes.POINTER(fopd_chunk), i32, vp, vp, fopd_params, vp, vp, vp, vp]
        L.fopd_loss_fwd_bwd_plan.argtypes = [i32, ctypes.c_int64] + [ctypes.POINTER(ctypes.c_int32)] * 4
        i64, f32 = ctypes.c_int64, ctypes.c_float
        L.fopd_loss_fwd_bwd_set_plan.argtypes = [i32, i64, i32]
        L.fopd_release_device_memory.argtypes = []
        L.fopd_selftest_bounded_wait.argtypes = [i64, vp, vp, vp]
        L.fopd_row_divergence.argtypes = [vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, vp, vp, vp, vp]
        L.fopd_supervision_drift.argtypes = [vp, vp, i32, vp, vp, vp, vp]
        L.fopd_refresh_decision.argtypes = [vp, vp, vp, i32, f32, f32, f32, i64, i64, vp, vp, vp]
        L.fopd_shard_stats.argtypes = [ctypes.POINTER(fopd_chunk), i64, i64, vp, vp]
        L.fopd_shard_merge.argtypes = [vp, i32, ctypes.POINTER(fopd_chunk), i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.fopd_shard_loss_fwd_bwd.argtypes = [ctypes.POINTER(fopd_chunk), i64, i64, i32, vp, vp, fopd_params, vp, vp,
                                              vp]
        L.fopd_loss_finalize.argtypes = [vp, vp, vp, i32, fopd_params, vp, vp, vp]
        L.fopd_check_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
        L.fopd_step_host_workspace_bytes.restype = ctypes.c_uint64
        L.fopd_step_host_workspace_bytes.argtypes = [ctypes.POINTER(fopd_chunk), i32, i32, i32]
        L.fopd_step_host.argtypes = [ctypes.POINTER(fopd_chunk), i32, i32, vp, vp, vp, fopd_params,
                                     ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(fopd_host_outputs), vp,
                                     ctypes.c_uint64, vp]
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().fopd_strerror(int(code)).decode()


def version() -> int:
    return int(lib().fopd_version())


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(rc: int, where: str):
    if rc != 0:
        raise FopdError(rc, where)


def params(alpha=1.0, beta=1.0, xi=0.15, lam=0.1) -> fopd_params:
    return fopd_params(float(alpha), float(beta), float(xi), float(lam))


@dataclass
class Chunk:
    """Device tensors of one chunk of token rows (see ``fopd_chunk`` in fopd.h)."""
    student: torch.Tensor  # [n, V] (row pitch = student.stride(0)), bf16 or fp32
    teacher: torch.Tensor | None  # None only for fopd_token_stats_student
    behav_logprob: torch.Tensor  # [n] fp32
    tokens: torch.Tensor  # [n] int32
    mask: torch.Tensor  # [n] uint8
    sample_id: torch.Tensor  # [n] int32
    vocab: int | None = None  # columns in use; defaults to student.shape[1]
    loss_kind: int = LOSS_FULL_KL

    def c_struct(self) -> fopd_chunk:
        S, T = self.student, self.teacher
        assert S.dtype in (torch.bfloat16, torch.float32) and S.dim() == 2 and S.stride(1) == 1
        assert T is None or (S.dtype == T.dtype and S.shape == T.shape and S.stride() == T.stride())
        assert self.behav_logprob.dtype == torch.float32 and self.tokens.dtype == torch.int32
        assert self.mask.dtype == torch.uint8 and self.sample_id.dtype == torch.int32
        n = S.shape[0]
        for t in (self.behav_logprob, self.tokens, self.mask, self.sample_id):
            assert t.is_contiguous() and t.numel() == n and t.device == S.device
        return fopd_chunk(
            S.data_ptr(), None if T is None else T.data_ptr(), self.behav_logprob.data_ptr(), self.tokens.data_ptr(),
            self.mask.data_ptr(), self.sample_id.data_ptr(), n, self.vocab or S.shape[1],
            S.stride(0) if n > 1 else max(S.stride(0), S.shape[1]),
            FOPD_BF16 if S.dtype == torch.bfloat16 else FOPD_F32, int(self.loss_kind),
        )


def fopd_token_stats(chunk: Chunk, B: int, acc, *, lp_s=None, lp_t=None, kl=None, ratio=None,
                     row_ws=None, status=None, stream=None):
    c = chunk.c_struct()
    _check(lib().fopd_token_stats(ctypes.byref(c), B, _ptr(lp_s), _ptr(lp_t), _ptr(kl), _ptr(ratio),
                                  _ptr(row_ws), _ptr(acc), _ptr(status), _stream(stream)),
           "fopd_token_stats")


def fopd_token_stats_student(chunk: Chunk, B: int, acc, *, lp_s=None, ratio=None, status=None, stream=None):
    """The student's half of fopd_token_stats (chunk.teacher may be None): enough for
    fopd_sample_freshness; the loss call that follows gets no row_ws."""
    c = chunk.c_struct()
    _check(lib().fopd_token_stats_student(ctypes.byref(c), B, _ptr(lp_s), _ptr(ratio), _ptr(acc), _ptr(status),
                                          _stream(stream)),
           "fopd_token_stats_student")


STATIC_MAX_ROWS = 65536
STATIC_MAX_SAMPLES = 16384


def fopd_token_stats_static(chunk: Chunk, B: int, acc, *, lp_s=None, lp_t=None, kl=None, ratio=None,
                            status=None, stream=None):
    """fopd_token_stats without any device allocation: the per-row scratch is a
    fixed 1 MiB array inside the library (at most STATIC_MAX_ROWS rows per call).
    For callers that have given all GPU memory to their own allocator or that
    forbid allocations inside their step loop.  Calls on one device share the
    scratch, so keep them on one stream."""
    c = chunk.c_struct()
    _check(lib().fopd_token_stats_static(ctypes.byref(c), B, _ptr(lp_s), _ptr(lp_t), _ptr(kl), _ptr(ratio),
                                         _ptr(acc), _ptr(status), _stream(stream)),
           "fopd_token_stats_static")


def fopd_sample_freshness(acc, staleness, seq_len, d_sup, B: int, p: fopd_params, *, coef, f=None,
                          w=None, d_roll=None, l_distill=None, m_align=None, buffer_means=None,
                          status=None, stream=None):
    _check(lib().fopd_sample_freshness(_ptr(acc), _ptr(staleness), _ptr(seq_len), _ptr(d_sup), B, p,
                                       _ptr(f), _ptr(w), _ptr(d_roll), _ptr(l_distill), _ptr(m_align),
                                       _ptr(coef), _ptr(buffer_means), _ptr(status), _stream(stream)),
           "fopd_sample_freshness")


def fopd_loss_fwd_bwd(chunk: Chunk, B: int, coef, p: fopd_params, dlogits, loss_acc, *, row_ws=None,
                      status=None, stream=None):
    c = chunk.c_struct()
    assert dlogits.dtype == chunk.student.dtype and dlogits.stride() == chunk.student.stride()
    _check(lib().fopd_loss_fwd_bwd(ctypes.byref(c), B, _ptr(coef), _ptr(row_ws), p, _ptr(dlogits),
                                   _ptr(loss_acc), _ptr(status), _stream(stream)),
           "fopd_loss_fwd_bwd")


def fopd_loss_fwd_bwd_plan(dtype: torch.dtype, vocab: int) -> dict:
    """Launch shape of fopd_loss_fwd_bwd(row_ws=None) on the current device (cluster_size 0:
    the streaming kernel pair is used instead)."""
    out = [ctypes.c_int32(0) for _ in range(4)]
    _check(lib().fopd_loss_fwd_bwd_plan(FOPD_BF16 if dtype == torch.bfloat16 else FOPD_F32, int(vocab),
                                        *[ctypes.byref(o) for o in out]), "fopd_loss_fwd_bwd_plan")
    return dict(zip(("cluster_size", "block_threads", "resident_clusters", "smem_bytes"),
                    (int(o.value) for o in out)))


def fopd_loss_fwd_bwd_set_plan(dtype: torch.dtype, vocab: int, cluster_size: int) -> None:
    """Pins the on-chip launch shape for (current device, dtype, vocab): cluster_size > 0 CTAs per
    cluster, < 0 the streaming kernel pair, 0 back to the library's own choice."""
    _check(lib().fopd_loss_fwd_bwd_set_plan(FOPD_BF16 if dtype == torch.bfloat16 else FOPD_F32, int(vocab),
                                            int(cluster_size)), "fopd_loss_fwd_bwd_set_plan")


def fopd_release_device_memory() -> None:
    """Trims the library's memory pool on the current device and drops fopd_step_host's streams."""
    _check(lib().fopd_release_device_memory(), "fopd_release_device_memory")


def fopd_selftest_bounded_wait(limit_cycles: int, status, waited_cycles=None, *, stream=None) -> None:
    """Runs one bounded barrier wait that cannot complete; the kernel sets the timeout bit in ``status``."""
    _check(lib().fopd_selftest_bounded_wait(int(limit_cycles), _ptr(status), _ptr(waited_cycles), _stream(stream)),
           "fopd_selftest_bounded_wait")


def fopd_loss_finalize(loss_acc, acc, w, B: int, p: fopd_params, loss_out, *, per_sample_loss=None,
                       stream=None):
    _check(lib().fopd_loss_finalize(_ptr(loss_acc), _ptr(acc), _ptr(w), B, p, _ptr(per_sample_loss),
                                    _ptr(loss_out), _stream(stream)),
           "fopd_loss_finalize")


def fopd_row_divergence(first, second, mask, sample_id, B: int, acc, *, kl=None, entropy=None, vocab=None,
                        status=None, stream=None):
    assert first.dtype == second.dtype and first.shape == second.shape and first.stride() == second.stride()
    n = first.shape[0]
    _check(lib().fopd_row_divergence(_ptr(first), _ptr(second), _ptr(mask), _ptr(sample_id), n,
                                     vocab or first.shape[1], first.stride(0) if n > 1 else first.shape[1],
                                     FOPD_BF16 if first.dtype == torch.bfloat16 else FOPD_F32, B, _ptr(kl),
                                     _ptr(entropy), _ptr(acc), _ptr(status), _stream(stream)),
           "fopd_row_divergence")


def fopd_supervision_drift(acc, seq_len, B: int, *, d_sup=None, m_sup=None, mean_entropy=None, stream=None):
    _check(lib().fopd_supervision_drift(_ptr(acc), _ptr(seq_len), B, _ptr(d_sup), _ptr(m_sup), _ptr(mean_entropy),
                                        _stream(stream)), "fopd_supervision_drift")


def fopd_refresh_decision(f, m_roll, m_sup, B: int, kappa_f, kappa_roll, kappa_sup, steps_since_refresh: int,
                          min_interval: int, decision, *, means=None, stream=None):
    _check(lib().fopd_refresh_decision(_ptr(f), _ptr(m_roll), _ptr(m_sup), B, float(kappa_f), float(kappa_roll),
                                       float(kappa_sup), int(steps_since_refresh), int(min_interval), _ptr(means),
                                       _ptr(decision), _stream(stream)), "fopd_refresh_decision")


def fopd_shard_stats(shard: Chunk, vocab_offset: int, vocab_total: int, partial, *, stream=None):
    """Partial sums [n_rows, 8] of the columns [vocab_offset, vocab_offset + W) held in ``shard``."""
    c = shard.c_struct()
    assert partial.dtype == torch.float32 and partial.is_contiguous() and partial.numel() == 8 * c.n_rows
    _check(lib().fopd_shard_stats(ctypes.byref(c), int(vocab_offset), int(vocab_total), _ptr(partial),
                                  _stream(stream)), "fopd_shard_stats")


def fopd_shard_merge(partials, behav_logprob, tokens, mask, sample_id, vocab_total: int, B: int, acc, row_ws, *,
                     lp_s=None, lp_t=None, kl=None, ratio=None, status=None, stream=None):
    """Merge of all parts ([n_parts, n_rows, 8]) into the row statistics and the per-sample sums."""
    n = tokens.numel()
    assert partials.dtype == torch.float32 and partials.is_contiguous() and partials.dim() == 3
    assert partials.shape[1] == n and partials.shape[2] == 8
    rows = fopd_chunk(None, None, behav_logprob.data_ptr(), tokens.data_ptr(), mask.data_ptr(),
                      sample_id.data_ptr(), n, int(vocab_total), int(vocab_total), FOPD_F32, LOSS_FULL_KL)
    _check(lib().fopd_shard_merge(_ptr(partials), partials.shape[0], ctypes.byref(rows), B, _ptr(lp_s), _ptr(lp_t),
                                  _ptr(kl), _ptr(ratio), _ptr(row_ws), _ptr(acc), _ptr(status), _stream(stream)),
           "fopd_shard_merge")


def fopd_shard_loss_fwd_bwd(shard: Chunk, vocab_offset: int, vocab_total: int, B: int, coef, row_ws,
                            p: fopd_params, dlogits, *, loss_acc=None, stream=None):
    c = shard.c_struct()
    assert dlogits.dtype == shard.student.dtype and dlogits.stride() == shard.student.stride()
    _check(lib().fopd_shard_loss_fwd_bwd(ctypes.byref(c), int(vocab_offset), int(vocab_total), B, _ptr(coef),
                                         _ptr(row_ws), p, _ptr(dlogits), _ptr(loss_acc), _stream(stream)),
           "fopd_shard_loss_fwd_bwd")


def fopd_check_status(status, stream=None) -> int:
    """Synchronises the stream and returns the device status bits (0 = clean)."""
    bits = ctypes.c_int32(0)
    rc = lib().fopd_check_status(_ptr(status), ctypes.byref(bits), _stream(stream))
    if rc not in (0, -8):
        raise FopdError(rc, "fopd_check_status")
    return int(bits.value)


def _chunk_array(chunks):
    arr = (fopd_chunk * len(chunks))()
    for j, ch in enumerate(chunks):
        arr[j] = ch.c_struct()
    return arr


def fopd_step_host_workspace_bytes(chunks, B: int, resident: bool) -> int:
    """Device workspace size fopd_step_host needs for these HOST chunks."""
    return int(lib().fopd_step_host_workspace_bytes(_chunk_array(chunks), len(chunks), B, int(resident)))


def fopd_step_host(chunks, B: int, staleness, seq_len, d_sup, p: fopd_params, dlogits, workspace, *,
                   stream=None) -> dict:
    """Whole batch from HOST tensors (``chunks`` hold CPU tensors, ideally pinned;
    ``dlogits`` is a list of CPU tensors receiving the gradients).  Returns the
    per-sample outputs as CPU tensors plus the scalar loss and status bits."""
    arr = _chunk_array(chunks)
    z = lambda n: torch.zeros(n, dtype=torch.float32)
    res = dict(f=z(B), w=z(B), d_roll=z(B), l_distill=z(B), m_align=z(B), per_sample_loss=z(B),
               buffer_means=z(2), loss=z(1), status_bits=torch.zeros(1, dtype=torch.int32),
               copied_bytes=torch.zeros(2, dtype=torch.int64))
    outs = fopd_host_outputs(*[res[n].data_ptr() for n, _ in fopd_host_outputs._fields_])
    dl = (ctypes.c_void_p * len(dlogits))(*[d.data_ptr() for d in dlogits])
    rc = lib().fopd_step_host(arr, len(chunks), B, _ptr(staleness), _ptr(seq_len), _ptr(d_sup), p, dl,
                              ctypes.byref(outs), _ptr(workspace), workspace.numel() * workspace.element_size(),
                              _stream(stream))
    if rc not in (0, -8):
        raise FopdError(rc, "fopd_step_host")
    return res
