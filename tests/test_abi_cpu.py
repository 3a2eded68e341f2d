"""CPU-side checks of the boundary: libfopd.so loads without a GPU, exports every
symbol include/fopd.h declares, and rejects bad arguments on the host before any
CUDA call.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_2605_17862_b200 import binding as fb
from paper_2605_17862_b200 import build as fbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fbuild.build_lib()
    return fb.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fopd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fopd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"fopd_token_stats", "fopd_sample_freshness", "fopd_loss_fwd_bwd"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in fopd.h but not exported"
    assert set(names) == set(fb.EXPORTS)
    assert fb.version() == 201


def test_strerror_covers_every_status(lib):
    seen = {fb.strerror(c) for c in range(0, -10, -1)}
    assert len(seen) == 10 and "unknown fopd status" not in seen
    assert fb.strerror(-99) == "unknown fopd status"


def _chunk(**kw):
    base = dict(student=0x1000, teacher=0x2000, behav_logprob=0x3000, tokens=0x4000, mask=0x5000,
                sample_id=0x6000, n_rows=4, vocab=64, row_stride=64, dtype=0, loss_kind=0)
    base.update(kw)
    return fb.fopd_chunk(*[base[f] for f, _ in fb.fopd_chunk._fields_])


@pytest.mark.parametrize("kw,code", [
    (dict(dtype=7), -4),
    (dict(loss_kind=2), -9),
    (dict(n_rows=-1), -3),
    (dict(vocab=0), -3),
    (dict(row_stride=32), -3),
    (dict(student=0), -1),
    (dict(tokens=0), -1),
    (dict(student=0x1008), -2),
    (dict(row_stride=68, vocab=60), -2),   # bf16 pitch of 136 bytes
])
def test_host_side_argument_checks(lib, kw, code):
    c = _chunk(**kw)
    acc = ctypes.c_void_p(0x7000)
    assert lib.fopd_token_stats(ctypes.byref(c), 2, None, None, None, None, None, acc, None, None) == code
    assert lib.fopd_token_stats_static(ctypes.byref(c), 2, None, None, None, None, acc, None, None) == code
    p = fb.params()
    assert lib.fopd_loss_fwd_bwd(ctypes.byref(c), 2, ctypes.c_void_p(0x8000), None, p,
                                 ctypes.c_void_p(0x100000), ctypes.c_void_p(0x9000), None, None) == code


def test_more_host_checks(lib):
    c = _chunk()
    p = fb.params()
    vp = ctypes.c_void_p
    assert lib.fopd_token_stats(None, 2, None, None, None, None, None, vp(0x7000), None, None) == -1
    assert lib.fopd_token_stats(ctypes.byref(c), 0, None, None, None, None, None, vp(0x7000), None, None) == -3
    assert lib.fopd_token_stats(ctypes.byref(c), 2, None, None, None, None, None, None, None, None) == -1
    assert lib.fopd_token_stats(ctypes.byref(c), 2, None, None, None, None, vp(0x7004), vp(0x7000), None, None) == -2
    # the student's half of the statistics: same checks, but the teacher is not needed
    no_teacher = _chunk(teacher=0)
    assert lib.fopd_token_stats(ctypes.byref(no_teacher), 2, None, None, None, None, None, vp(0x7000), None, None) == -1
    assert lib.fopd_token_stats_student(ctypes.byref(no_teacher), 2, None, None, None, None, None) == -1   # acc
    assert lib.fopd_token_stats_student(ctypes.byref(_chunk(teacher=0, student=0)), 2, None, None, vp(0x7000), None, None) == -1
    assert lib.fopd_token_stats_student(ctypes.byref(_chunk(teacher=0, student=0x1008)), 2, None, None, vp(0x7000), None, None) == -2
    assert lib.fopd_token_stats_student(ctypes.byref(_chunk(teacher=0, n_rows=0)), 2, None, None, vp(0x7000), None, None) == 0
    assert lib.fopd_token_stats_student(ctypes.byref(_chunk(teacher=0, dtype=5)), 2, None, None, vp(0x7000), None, None) == -4
    big = _chunk(n_rows=fb.STATIC_MAX_ROWS + 1)
    assert lib.fopd_token_stats_static(ctypes.byref(big), 2, None, None, None, None, vp(0x7000), None, None) == -3
    # empty chunk: nothing to do, no CUDA call
    empty = _chunk(n_rows=0, student=0, teacher=0)
    assert lib.fopd_token_stats(ctypes.byref(empty), 2, None, None, None, None, None, vp(0x7000), None, None) == 0
    # parameters
    for bad in (fb.params(alpha=-1), fb.params(beta=-0.5), fb.params(xi=float("nan")), fb.params(lam=float("inf"))):
        assert lib.fopd_sample_freshness(vp(8), vp(8), vp(8), None, 2, bad, None, None, None, None, None, vp(8),
                                         None, None, None) == -5
        assert lib.fopd_loss_finalize(vp(8), vp(8), vp(8), 2, bad, None, vp(8), None) == -5
    assert lib.fopd_sample_freshness(vp(8), vp(8), vp(8), None, 2, p, None, None, None, None, None, None,
                                     None, None, None) == -1
    assert lib.fopd_sample_freshness(vp(8), vp(8), vp(8), None, 0, p, None, None, None, None, None, vp(8),
                                     None, None, None) == -3
    # dlogits overlapping the student rows
    assert lib.fopd_loss_fwd_bwd(ctypes.byref(c), 2, vp(0x8000), None, p, vp(0x1100), vp(0x9000), None, None) == -7
    assert lib.fopd_check_status(None, None, None) == -1
    # host-buffer entry: workspace sizes grow with residency, bad chunk gives 0
    hc = _chunk(n_rows=1000, vocab=1024, row_stride=1024)
    arr = (fb.fopd_chunk * 2)(hc, hc)
    small = lib.fopd_step_host_workspace_bytes(arr, 2, 4, 0)
    large = lib.fopd_step_host_workspace_bytes(arr, 2, 4, 1)
    assert 3 * 1000 * 1024 * 2 <= small < large and large >= 5 * 1000 * 1024 * 2
    assert lib.fopd_step_host_workspace_bytes((fb.fopd_chunk * 1)(_chunk(dtype=9)), 1, 4, 0) == 0


def test_shard_entry_points_check_arguments_on_the_host(lib):
    vp = ctypes.c_void_p
    p = fb.params()
    sh = _chunk(vocab=32, row_stride=64)  # columns [v0, v0 + 32) of rows with a pitch of 64
    part, ws, coef, acc, out = vp(0x7000), vp(0x8000), vp(0x9000), vp(0xa000), vp(0x100000)
    assert lib.fopd_shard_stats(ctypes.byref(sh), -8, 64, part, None) == -3            # negative offset
    assert lib.fopd_shard_stats(ctypes.byref(sh), 40, 64, part, None) == -3            # reaches past the vocabulary
    assert lib.fopd_shard_stats(ctypes.byref(sh), 0, (1 << 30) + 1, part, None) == -3
    assert lib.fopd_shard_stats(ctypes.byref(sh), 0, 64, None, None) == -1
    assert lib.fopd_shard_stats(ctypes.byref(sh), 0, 64, vp(0x7004), None) == -2
    assert lib.fopd_shard_stats(ctypes.byref(_chunk(student=0x1008, vocab=32)), 0, 64, part, None) == -2
    assert lib.fopd_shard_stats(None, 0, 64, part, None) == -1
    assert lib.fopd_shard_stats(ctypes.byref(_chunk(n_rows=0, student=0, teacher=0, vocab=32)), 0, 64, None, None) == 0
    rows = _chunk(student=0, teacher=0, vocab=64)  # the merge ignores the logits pointers
    assert lib.fopd_shard_merge(part, 0, ctypes.byref(rows), 2, None, None, None, None, ws, acc, None, None) == -3
    assert lib.fopd_shard_merge(part, 2, ctypes.byref(rows), 2, None, None, None, None, None, acc, None, None) == -1
    assert lib.fopd_shard_merge(part, 2, ctypes.byref(rows), 2, None, None, None, None, ws, None, None, None) == -1
    assert lib.fopd_shard_merge(None, 2, ctypes.byref(rows), 2, None, None, None, None, ws, acc, None, None) == -1
    assert lib.fopd_shard_merge(part, 2, ctypes.byref(_chunk(tokens=0)), 2, None, None, None, None, ws, acc, None,
                                None) == -1
    assert lib.fopd_shard_merge(part, 2, ctypes.byref(rows), 0, None, None, None, None, ws, acc, None, None) == -3
    assert lib.fopd_shard_merge(part, 2, ctypes.byref(rows), 2, None, None, None, None, vp(0x8004), acc, None,
                                None) == -2
    f = lib.fopd_shard_loss_fwd_bwd
    assert f(ctypes.byref(sh), 0, 64, 2, coef, None, p, out, None, None) == -1        # merged statistics required
    assert f(ctypes.byref(sh), 0, 64, 2, None, ws, p, out, None, None) == -1
    assert f(ctypes.byref(sh), 0, 64, 2, coef, ws, p, None, None, None) == -1
    assert f(ctypes.byref(sh), 40, 64, 2, coef, ws, p, out, None, None) == -3
    assert f(ctypes.byref(sh), 0, 64, 0, coef, ws, p, out, None, None) == -3
    assert f(ctypes.byref(sh), 0, 64, 2, coef, ws, fb.params(alpha=-1), out, None, None) == -5
    assert f(ctypes.byref(sh), 0, 64, 2, coef, ws, p, vp(0x1010), None, None) == -7     # over the student's columns


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(fb, "_lib", None)
    monkeypatch.setattr(fb, "LIB_PATH", str(tmp_path / "libfopd.so"))
    with pytest.raises(FileNotFoundError):
        fb.lib()


def test_new_control_entry_points_check_their_arguments_on_the_host(lib):
    """No GPU: these return before any CUDA call."""
    assert lib.fopd_loss_fwd_bwd_set_plan(7, 151936, 4) == -4          # dtype
    assert lib.fopd_loss_fwd_bwd_set_plan(0, 0, 4) == -3               # vocabulary
    assert lib.fopd_loss_fwd_bwd_set_plan(0, 151936, 17) == -3         # more CTAs than a cluster can have
    assert lib.fopd_selftest_bounded_wait(1000, None, None, None) == -1
    status = ctypes.c_void_p(0x1000)
    assert lib.fopd_selftest_bounded_wait(-1, status, None, None) == -3
    assert lib.fopd_selftest_bounded_wait(10**12, status, None, None) == -3
