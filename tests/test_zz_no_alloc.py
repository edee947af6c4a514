"""The allocation-free scorer (focus_score_blocks_static) against the regular entry point and against the oracle.

Some users of this library are not allowed to allocate on the GPU at all -- they run inside a server whose
memory pool owns the device, or on a path where cudaMalloc's device-wide synchronisation would stall other work --
so they can neither create a context nor let the library grab scratch.  For them the library carries one
context-free entry point whose scratch is a fixed array compiled into it.  This file (collected last) checks,
through the C ABI, that it returns what focus_score_blocks returns and what the CPU oracle computes (Eq. 7), twice
in a row (the array is shared between calls and keeps old contents), in both head modes, warm and cold, with and
without a caller-owned status word; that it works in a process that never created a context; that shapes exactly at
the limits of the fixed scratch are taken and shapes beyond them are refused instead of overrunning it."""
import ctypes as C
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2602_02159_b200 import binding as fb
from paper_2602_02159_b200 import step as fstep
from paper_2602_02159_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FOCUS_POS = [1101, 1110, 1133, 1190, 1200]


def _inputs(dtype, H, Hkv, d, B, seed):
    s = wl.Shape(1500, 1100, H, Hkv, d, B, dtype)
    t = wl.gen_qkv(s, seed, threads=2)
    dQ, dK = fstep.to_device(t["Q"], dtype), fstep.to_device(t["K"], dtype)
    focus = torch.tensor(FOCUS_POS + [-1, -1, -1], dtype=torch.int32, device="cuda")
    n_focus = torch.tensor([len(FOCUS_POS)], dtype=torch.int32, device="cuda")
    return s, t, dQ, dK, focus, n_focus


def _oracle_R(s, t, focus_pos, head_reduce):
    """Eq. 7 by the oracle, one KV group at a time (bounds host memory at the large shapes)."""
    hpg = s.H // s.Hkv
    rows = np.asarray(focus_pos) - s.M
    per_group = np.zeros((s.Hkv, s.nb))
    for g in range(s.Hkv):
        Kg = wl.storage_to_f64(t["K"][g:g + 1], s.dtype)
        Qg = wl.storage_to_f64(t["Q"][rows][:, g * hpg:(g + 1) * hpg], s.dtype)
        per_group[g] = fo.score_blocks(Qg, fo.pool_keys(Kg, s.M, s.B), fo.PER_KV_GROUP)[0]
    if head_reduce == fb.HEADS_ALL:                    # equal group sizes: the mean over heads is the mean of group means
        return per_group.mean(axis=0, keepdims=True)
    return per_group


@pytest.mark.parametrize("cfg", [("bf16", 8, 2, 128, 128), ("f32", 4, 4, 64, 64)])
def test_static_scorer_matches_regular_entry_point_and_oracle_twice_in_a_row(cfg):
    dtype, H, Hkv, d, B = cfg
    ctx = fb.Context(0)
    for call, seed in enumerate((21, 22)):             # two calls in a row, different data: no stale scratch may leak
        s, t, dQ, dK, focus, n_focus = _inputs(dtype, H, Hkv, d, B, seed)
        sh = fstep.c_shape(s)
        Kbar = torch.zeros(Hkv, s.nb, d, dtype=torch.float32, device="cuda")
        fb.focus_pool_keys(ctx, sh, dK, Kbar)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for head_reduce in (fb.HEADS_PER_KV_GROUP, fb.HEADS_ALL):
            G = Hkv if head_reduce == fb.HEADS_PER_KV_GROUP else 1
            R_ora = _oracle_R(s, t, FOCUS_POS, head_reduce).reshape(-1)
            for warm in (True, False):
                for own_status in (True, False):       # False: the status word inside the library's fixed array
                    ref = torch.zeros(G * s.nb, dtype=torch.float32, device="cuda")
                    got = torch.full((G * s.nb,), 7.0, dtype=torch.float32, device="cuda")
                    fb.focus_score_blocks(ctx, sh, dQ, s.M, focus, n_focus, 8, None if warm else dK,
                                          Kbar if warm else None, head_reduce, ref)
                    fb.focus_score_blocks_static(sh, dQ, s.M, focus, n_focus, 8, None if warm else dK,
                                                 Kbar if warm else None, head_reduce, got,
                                                 status if own_status else None)
                    torch.cuda.synchronize()
                    scale = max(1.0, float(ref.abs().max()))
                    assert float((got - ref).abs().max()) <= 1e-5 * scale, (call, head_reduce, warm)
                    assert float(np.abs(got.cpu().numpy().astype(np.float64) - R_ora).max()) <= 1e-5 * scale, \
                        (call, head_reduce, warm)
                    assert float(ref.abs().max()) > 0
        assert status.item() == 0 and ctx.poll_status() == 0
    ctx.close()


def test_static_scorer_in_a_process_that_never_created_a_context():
    """The stated use: no focus_create anywhere in the process, the very first library call is the static scorer."""
    code = textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        import numpy as np, torch
        from oracle import focus_oracle as fo
        from paper_2602_02159_b200 import binding as fb, step as fstep, workloads as wl
        s = wl.Shape(900, 700, 4, 2, 128, 64, "bf16")
        t = wl.gen_qkv(s, 31, threads=1)
        dQ, dK = fstep.to_device(t["Q"], "bf16"), fstep.to_device(t["K"], "bf16")
        pos = [700, 731, 899]
        focus = torch.tensor(pos + [-1], dtype=torch.int32, device="cuda")
        n_focus = torch.tensor([3], dtype=torch.int32, device="cuda")
        Q, K = wl.storage_to_f64(t["Q"], "bf16"), wl.storage_to_f64(t["K"], "bf16")
        R_ora = fo.score_blocks(Q[np.array(pos) - s.M], fo.pool_keys(K, s.M, s.B), fo.PER_KV_GROUP).reshape(-1)
        for _ in range(2):
            R = torch.full((s.Hkv * s.nb,), 3.0, dtype=torch.float32, device="cuda")
            fb.focus_score_blocks_static(fstep.c_shape(s), dQ, s.M, focus, n_focus, 4, dK, None, 0, R, None)
            torch.cuda.synchronize()
            err = float(np.abs(R.cpu().numpy().astype(np.float64) - R_ora).max())
            assert err <= 1e-5 * max(1.0, float(np.abs(R_ora).max())), err
        print("static-only process ok")
        """ % ROOT)
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "static-only process ok" in r.stdout, r.stdout + r.stderr


def test_static_scorer_takes_shapes_exactly_at_its_limits():
    """n_kv_heads * head_dim = 8192 and, in all-heads mode, n_kv_heads * nb = 65536: both fit the fixed array exactly."""
    s = wl.Shape(512 * 64 + 64, 512 * 64, 128, 128, 64, 64, "bf16")
    assert s.Hkv * s.d == 8192 and s.Hkv * s.nb == 65536
    t = wl.gen_qkv(s, 41)
    dQ, dK = fstep.to_device(t["Q"], "bf16"), fstep.to_device(t["K"], "bf16")
    pos = [s.M, s.M + 7, s.M + 63]
    focus = torch.tensor(pos, dtype=torch.int32, device="cuda")
    n_focus = torch.tensor([3], dtype=torch.int32, device="cuda")
    sh = fstep.c_shape(s)
    for head_reduce in (fb.HEADS_ALL, fb.HEADS_PER_KV_GROUP):
        G = 1 if head_reduce == fb.HEADS_ALL else s.Hkv
        R = torch.zeros(G * s.nb, dtype=torch.float32, device="cuda")
        fb.focus_score_blocks_static(sh, dQ, s.M, focus, n_focus, 3, dK, None, head_reduce, R, None)
        torch.cuda.synchronize()
        R_ora = _oracle_R(s, t, pos, head_reduce).reshape(-1)
        assert float(np.abs(R.cpu().numpy().astype(np.float64) - R_ora).max()) <= 1e-5 * max(1.0, np.abs(R_ora).max())
    # one step past either limit is refused before anything is launched
    lib = fb.load_library()
    st = torch.cuda.current_stream().cuda_stream
    p = lambda x: x.data_ptr()
    R = torch.zeros(s.Hkv * (s.nb + 1), dtype=torch.float32, device="cuda")
    past_nb = fb.make_shape(s.L + 64, s.M + 1, s.H, s.Hkv, s.d, s.B, fb.BF16)          # nb = 513: 128 * 513 > 65536
    assert lib.focus_score_blocks_static(C.byref(past_nb), p(dQ), s.M + 1, p(focus), p(n_focus), 3, p(dK), None,
                                         fb.HEADS_ALL, p(R), None, st) == fb.ERR_WORKSPACE_TOO_SMALL
    past_qbar = fb.make_shape(s.L, s.M, 136, 136, s.d, s.B, fb.BF16)                   # 136 * 64 > 8192
    assert lib.focus_score_blocks_static(C.byref(past_qbar), p(dQ), s.M, p(focus), p(n_focus), 3, p(dK), None,
                                         fb.HEADS_PER_KV_GROUP, p(R), None, st) == fb.ERR_WORKSPACE_TOO_SMALL


def test_static_scorer_rejects_what_does_not_fit_and_reports_anomalies():
    lib = fb.load_library()
    s, _, dQ, dK, focus, n_focus = _inputs("bf16", 8, 2, 128, 128, 23)
    R = torch.zeros(8 * 4096, dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    p = lambda t: t.data_ptr()
    # n_kv_heads * head_dim beyond the fixed scratch (128 KV heads x 128)
    big = fb.make_shape(1500, 1100, 128, 128, 128, 128, fb.BF16)
    assert lib.focus_score_blocks_static(C.byref(big), p(dQ), 1100, p(focus), p(n_focus), 8, p(dK), None, 0, p(R), None,
                                         st) == fb.ERR_WORKSPACE_TOO_SMALL
    # all-heads mode with more (KV heads x blocks) than fit: 64 KV heads, 2M prompt tokens in 64-token blocks
    wide = fb.make_shape(2_200_000, 2_100_000, 64, 64, 128, 64, fb.BF16)
    assert lib.focus_score_blocks_static(C.byref(wide), p(dQ), 2_100_000, p(focus), p(n_focus), 8, p(dK), None, 1,
                                         p(R), None, st) == fb.ERR_WORKSPACE_TOO_SMALL
    # neither / both of K and Kbar
    sh = fstep.c_shape(s)
    assert lib.focus_score_blocks_static(C.byref(sh), p(dQ), s.M, p(focus), p(n_focus), 8, None, None, 0, p(R), None,
                                         st) == fb.ERR_INVALID_ARG
    # a focus index outside the rows of Q is skipped and reported through the caller's status word
    bad = focus.clone()
    bad[1] = 5
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    fb.focus_score_blocks_static(sh, dQ, s.M, bad, n_focus, 8, dK, None, 0, R, status)
    torch.cuda.synchronize()
    assert status.item() == fb.ERR_INVALID_ARG
