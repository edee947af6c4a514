"""The allocation-free scorer (focus_score_blocks_static) against the regular entry point.

Some users of this library are not allowed to allocate on the GPU at all -- they run inside a server whose
memory pool owns the device, or on a path where cudaMalloc's device-wide synchronisation would stall other work --
so they can neither create a context nor let the library grab scratch.  For them the library carries one
context-free entry point whose scratch is a fixed array compiled into it.  This file (collected last) checks,
through the C ABI, that it returns what focus_score_blocks returns, twice in a row (the array is shared between
calls and keeps old contents), in both head modes, warm and cold, and that it refuses shapes beyond its fixed
scratch instead of overrunning it."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2602_02159_b200 import binding as fb
from paper_2602_02159_b200 import step as fstep
from paper_2602_02159_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _inputs(dtype, H, Hkv, d, B, seed):
    s = wl.Shape(1500, 1100, H, Hkv, d, B, dtype)
    t = wl.gen_qkv(s, seed, threads=2)
    dQ, dK = fstep.to_device(t["Q"], dtype), fstep.to_device(t["K"], dtype)
    focus = torch.tensor([1101, 1110, 1133, 1190, 1200, -1, -1, -1], dtype=torch.int32, device="cuda")
    n_focus = torch.tensor([5], dtype=torch.int32, device="cuda")
    return s, dQ, dK, focus, n_focus


@pytest.mark.parametrize("cfg", [("bf16", 8, 2, 128, 128), ("f32", 4, 4, 64, 64)])
def test_static_scorer_matches_regular_entry_point_twice_in_a_row(cfg):
    dtype, H, Hkv, d, B = cfg
    ctx = fb.Context(0)
    for call, seed in enumerate((21, 22)):             # two calls in a row, different data: no stale scratch may leak
        s, dQ, dK, focus, n_focus = _inputs(dtype, H, Hkv, d, B, seed)
        sh = fstep.c_shape(s)
        Kbar = torch.zeros(Hkv, s.nb, d, dtype=torch.float32, device="cuda")
        fb.focus_pool_keys(ctx, sh, dK, Kbar)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for head_reduce in (fb.HEADS_PER_KV_GROUP, fb.HEADS_ALL):
            G = Hkv if head_reduce == fb.HEADS_PER_KV_GROUP else 1
            for warm in (True, False):
                ref = torch.zeros(G * s.nb, dtype=torch.float32, device="cuda")
                got = torch.full((G * s.nb,), 7.0, dtype=torch.float32, device="cuda")
                fb.focus_score_blocks(ctx, sh, dQ, s.M, focus, n_focus, 8, None if warm else dK,
                                      Kbar if warm else None, head_reduce, ref)
                fb.focus_score_blocks_static(sh, dQ, s.M, focus, n_focus, 8, None if warm else dK,
                                             Kbar if warm else None, head_reduce, got, status)
                torch.cuda.synchronize()
                scale = max(1.0, float(ref.abs().max()))
                assert float((got - ref).abs().max()) <= 1e-5 * scale, (call, head_reduce, warm)
                assert float(ref.abs().max()) > 0
        assert status.item() == 0 and ctx.poll_status() == 0
    ctx.close()


def test_static_scorer_rejects_what_does_not_fit_and_reports_anomalies():
    lib = fb.load_library()
    s, dQ, dK, focus, n_focus = _inputs("bf16", 8, 2, 128, 128, 23)
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
