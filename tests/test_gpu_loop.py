"""GPU parity of the two loop-closing stages: confidence from logits (Eq. 2) and the KV-cache refresh (Eq. 3)."""
import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2602_02159_b200 import binding as fb
from paper_2602_02159_b200 import step as fstep
from paper_2602_02159_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = fb.Context(0)
    yield c
    assert c.poll_status() == 0
    c.close()


@pytest.mark.parametrize("dtype,vocab,stride", [("bf16", 126464, 126464), ("f32", 50257, 50260), ("bf16", 1003, 1008),
                                                ("f32", 7, 8)])
def test_confidence_against_oracle(ctx, dtype, vocab, stride):
    rng = np.random.default_rng(vocab)
    n_pos, pos_base = 96, 1000
    x = (rng.standard_normal((n_pos, stride)) * 3.0).astype(np.float32)
    x[3, 5 % vocab] = np.nan                                        # a NaN logit never wins
    x[4, :vocab] = 1.25                                             # a fully tied row: token 0, confidence 1/V
    xs = wl.to_storage(x, dtype)
    xf = wl.storage_to_f64(xs, dtype)[:, :vocab]
    dx = fstep.to_device(xs, dtype)
    rows_np = np.array(sorted(rng.choice(n_pos, size=40, replace=False)) + [-1] * 8, dtype=np.int32)
    rows_np[:40] += pos_base
    rows = torch.from_numpy(rows_np).cuda()
    n_rows = torch.tensor([40], dtype=torch.int32, device="cuda")
    conf = torch.full((48,), 7.0, dtype=torch.float32, device="cuda")
    tok = torch.full((48,), 7, dtype=torch.int32, device="cuda")
    fb.focus_confidence(ctx, dx, fb.BF16 if dtype == "bf16" else fb.F32, stride, vocab, pos_base, n_pos, rows, n_rows, 48,
                        conf, tok)
    ec, et = fo.confidence(xf[rows_np[:40] - pos_base])
    gc, gt = conf.cpu().numpy(), tok.cpu().numpy()
    assert gt[:40].tolist() == et.tolist()
    assert np.max(np.abs(gc[:40] - ec) / ec) < 1e-4
    assert (gt[40:] == -1).all() and (gc[40:] == 0).all()
    # all rows, no list
    conf2 = torch.zeros(n_pos, dtype=torch.float32, device="cuda")
    tok2 = torch.zeros(n_pos, dtype=torch.int32, device="cuda")
    fb.focus_confidence(ctx, dx, fb.BF16 if dtype == "bf16" else fb.F32, stride, vocab, pos_base, n_pos, None, None, n_pos,
                        conf2, tok2)
    ec, et = fo.confidence(xf)
    assert tok2.cpu().numpy().tolist() == et.tolist()
    assert np.max(np.abs(conf2.cpu().numpy() - ec) / ec) < 1e-4
    assert et[4] == 0 and abs(conf2[4].item() - 1.0 / vocab) < 1e-4 / vocab * 10
    assert ctx.poll_status() == 0


def test_confidence_feeds_the_indicator_and_the_unmasking(ctx):
    """conf^(t) from logits -> (a) top-n unmasking = the selection call with k = n, w = 0; (b) next step's focus set."""
    rng = np.random.default_rng(5)
    L, M, V = 640, 512, 4096
    logits = wl.to_storage((rng.standard_normal((L - M, V)) * 2).astype(np.float32), "bf16")
    d_logits = fstep.to_device(logits, "bf16")
    conf_full = torch.zeros(L, dtype=torch.float32, device="cuda")
    tok = torch.zeros(L - M, dtype=torch.int32, device="cuda")
    fb.focus_confidence(ctx, d_logits, fb.BF16, V, V, M, L - M, None, None, L - M, conf_full[M:], tok)
    masked = np.zeros(L, dtype=np.uint8)
    masked[M:M + 64] = (rng.random(64) < 0.7)
    dm = torch.from_numpy(masked).cuda()
    for k, w in ((2, 0), (8, 8)):
        f = torch.zeros(k, dtype=torch.int32, device="cuda"); nf = torch.zeros(1, dtype=torch.int32, device="cuda")
        a = torch.zeros(k * (2 * (w // 2) + 1), dtype=torch.int32, device="cuda"); na = torch.zeros(1, dtype=torch.int32, device="cuda")
        fb.focus_select_queries(ctx, conf_full, dm, L, M, M + 32, k, w, M, L, f, nf, a, na)
        ef, ea = fo.select_queries(conf_full.cpu().numpy(), masked, M, M + 32, k, w, M, L)
        assert f.cpu().numpy()[:nf.item()].tolist() == ef.tolist() and a.cpu().numpy()[:na.item()].tolist() == ea.tolist()
    ec, et = fo.confidence(wl.storage_to_f64(logits, "bf16"))
    assert tok.cpu().numpy().tolist() == et.tolist()
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("dtype,d,Hkv", [("bf16", 128, 4), ("f32", 64, 2), ("f32", 128, 1)])
def test_update_kv_bit_exact(ctx, dtype, d, Hkv):
    rng = np.random.default_rng(d)
    s = wl.Shape(700, 600, Hkv * 2, Hkv, d, 64, dtype)
    K = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    V = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    Kn = wl.to_storage(rng.standard_normal((40, Hkv, d)).astype(np.float32), dtype)
    Vn = wl.to_storage(rng.standard_normal((40, Hkv, d)).astype(np.float32), dtype)
    pos = np.sort(rng.choice(np.arange(600, 700), size=30, replace=False)).astype(np.int32)
    rows = torch.from_numpy(np.concatenate([pos, np.full(10, -1, dtype=np.int32)])).cuda()
    n_rows = torch.tensor([30], dtype=torch.int32, device="cuda")
    dK, dV = fstep.to_device(K, dtype), fstep.to_device(V, dtype)
    fb.focus_update_kv(ctx, fstep.c_shape(s), dK, dV, fstep.to_device(Kn, dtype), fstep.to_device(Vn, dtype), rows, n_rows, 40)
    eK, eV = fo.update_kv(K, V, Kn[:30], Vn[:30], pos)
    view = (lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)) if dtype == "bf16" else (lambda t: t.cpu().numpy())
    assert np.array_equal(view(dK), eK) and np.array_equal(view(dV), eV)
    assert ctx.poll_status() == 0
    # an out-of-range position is skipped and reported
    rows[0] = s.L + 5
    fb.focus_update_kv(ctx, fstep.c_shape(s), dK, dV, fstep.to_device(Kn, dtype), fstep.to_device(Vn, dtype), rows, n_rows, 40)
    assert ctx.poll_status() == fb.ERR_INVALID_ARG


@pytest.mark.gpu
def test_stream_read_probe_checksum_is_exact(ctx):
    """The read-only streaming probe xors every 32-bit word it reads: compared bit for bit with numpy on sizes
    below one vector per thread, with a ragged tail of the unrolled loop, and of several grid strides."""
    rng = np.random.default_rng(5)
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    for n_words in (0, 4, 4 * 1000, 4 * (148 * 8 * 256 * 8 + 12345), 4 * 3_000_001):
        host = rng.integers(0, 2 ** 32, size=n_words, dtype=np.uint32)
        dev = torch.from_numpy(host.view(np.int32)).cuda() if n_words else torch.zeros(4, dtype=torch.int32, device="cuda")
        fb.focus_stream_read(ctx, dev, n_words * 4, out)
        torch.cuda.synchronize()
        want = int(np.bitwise_xor.reduce(host)) if n_words else 0
        assert int(out.cpu().numpy().view(np.uint32)[0]) == want
    with pytest.raises(fb.FocusError):
        fb.focus_stream_read(ctx, dev, 24, out)                     # not a multiple of 16 bytes
    assert ctx.poll_status() == 0


# ---- end of a step on the device: new confidences in, the n most confident masked positions out -------------------
@pytest.mark.parametrize("mode", ["row_list", "all_positions", "ties_and_nan", "long_list"])
def test_commit_step_bit_exact(ctx, mode):
    rng = np.random.default_rng({"row_list": 1, "all_positions": 2, "ties_and_nan": 3, "long_list": 4}[mode])
    L, M = (9000, 5000) if mode == "long_list" else (900, 500)
    conf = rng.random(L).astype(np.float32)
    masked = np.zeros(L, dtype=np.uint8)
    masked[M:] = rng.random(L - M) < 0.7
    x = rng.integers(1, 30000, size=L).astype(np.int32)
    x[masked != 0] = 0
    if mode == "all_positions":                       # rows = NULL: positions pos_base .. pos_base + max_rows - 1
        pos = np.arange(M, M + 300)
        max_rows, n = 300, 300
    elif mode == "long_list":
        pos = np.sort(rng.choice(np.arange(M, L), size=4000, replace=False))
        max_rows, n = 4096, 4000
    else:
        pos = np.sort(rng.choice(np.arange(M - 10, L), size=70, replace=False))
        max_rows, n = 96, 70
    cn = rng.random(n).astype(np.float32)
    if mode in ("ties_and_nan", "long_list"):
        cn = (np.round(cn * 16) / 16).astype(np.float32)
        cn[rng.integers(0, n, size=3)] = np.nan
        cn[rng.integers(0, n, size=3)] = -0.0
    tn = rng.integers(1, 30000, size=n).astype(np.int32)
    blk_lo, blk_hi = (M, L) if mode == "long_list" else (M + 16, M + 200)
    for n_unmask in (0, 1, 2, 7, 600 if mode == "long_list" else 40):
        d_conf, d_masked, d_x = (torch.from_numpy(a.copy()).cuda() for a in (conf, masked, x))
        pad = lambda a, fill: np.concatenate([a, np.full(max_rows - n, fill, dtype=a.dtype)])
        d_cn, d_tn = torch.from_numpy(pad(cn, 9.0)).cuda(), torch.from_numpy(pad(tn, -5)).cuda()
        d_rows = None if mode == "all_positions" else torch.from_numpy(pad(pos.astype(np.int32), -1)).cuda()
        d_n = None if mode == "all_positions" else torch.tensor([n], dtype=torch.int32, device="cuda")
        out = torch.full((max(1, n_unmask),), -7, dtype=torch.int32, device="cuda")
        n_out = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        fb.focus_commit_step(ctx, d_cn, d_tn, M, d_rows, d_n, max_rows, L, blk_lo, blk_hi, n_unmask, d_conf, d_masked,
                             d_x, out, n_out)
        ec, em, ex, picks = fo.commit_step(conf, masked, x, pos.tolist(), cn, tn, blk_lo, blk_hi, n_unmask)
        assert n_out.item() == len(picks)
        got = out.cpu().numpy()
        assert got[:len(picks)].tolist() == picks and (n_unmask == 0 or (got[len(picks):n_unmask] == -1).all())
        assert np.array_equal(d_conf.cpu().numpy().view(np.uint32), ec.astype(np.float32).view(np.uint32))
        assert np.array_equal(d_masked.cpu().numpy(), em) and np.array_equal(d_x.cpu().numpy(), ex)
    assert ctx.poll_status() == 0
    # a position outside [0, L) is skipped and reported; bad host arguments are refused before any launch
    if mode == "row_list":
        bad = torch.from_numpy(pad(pos.astype(np.int32), -1)).cuda()
        bad[3] = L + 4
        fb.focus_commit_step(ctx, d_cn, d_tn, M, bad, d_n, max_rows, L, blk_lo, blk_hi, 2, d_conf, d_masked, d_x, out, n_out)
        assert ctx.poll_status() == fb.ERR_INVALID_ARG
        with pytest.raises(fb.FocusError):
            fb.focus_commit_step(ctx, d_cn, d_tn, M, bad, d_n, 5000, L, blk_lo, blk_hi, 2, d_conf, d_masked, d_x, out, n_out)
        with pytest.raises(fb.FocusError):
            fb.focus_commit_step(ctx, d_cn, d_tn, M, bad, None, 96, L, blk_lo, blk_hi, 2, d_conf, d_masked, d_x, out, n_out)


@pytest.mark.parametrize("dtype,d,B,Hkv", [("bf16", 128, 128, 4), ("bf16", 128, 64, 2), ("f32", 64, 64, 2)])
def test_pooled_keys_follow_a_cache_refresh(ctx, dtype, d, B, Hkv):
    """focus_update_kv of some prompt rows (as at a block-entry refresh) + focus_update_pooled_keys of the same rows
    = pooling the refreshed cache from scratch, bit for bit; and both equal the oracle's pooling of the refreshed
    cache.  The prompt length is not a multiple of the block size (short last block, refreshed too)."""
    rng = np.random.default_rng(B + d)
    s = wl.Shape(1500, 1100, Hkv * 2, Hkv, d, B, dtype)
    K = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    V = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    n, max_rows = 37, 48
    pos = np.sort(np.concatenate([rng.choice(np.arange(0, 1090), size=n - 5, replace=False), [1095, 1099],
                                  [1100, 1250, 1499]])).astype(np.int32)       # prompt rows, the short tail, 3 response rows
    Kn = wl.to_storage(rng.standard_normal((max_rows, Hkv, d)).astype(np.float32) * 3, dtype)
    Vn = wl.to_storage(rng.standard_normal((max_rows, Hkv, d)).astype(np.float32), dtype)
    rows = torch.from_numpy(np.concatenate([pos, np.full(max_rows - n, -1, dtype=np.int32)])).cuda()
    n_rows = torch.tensor([n], dtype=torch.int32, device="cuda")
    sh = fstep.c_shape(s)
    dK, dV = fstep.to_device(K, dtype), fstep.to_device(V, dtype)
    Kbar = torch.zeros(Hkv, s.nb, d, dtype=torch.float32, device="cuda")
    fb.focus_pool_keys(ctx, sh, dK, Kbar)
    before = Kbar.clone()
    fb.focus_update_kv(ctx, sh, dK, dV, fstep.to_device(Kn, dtype), fstep.to_device(Vn, dtype), rows, n_rows, max_rows)
    fb.focus_update_pooled_keys(ctx, sh, dK, Kbar, rows, n_rows, max_rows)
    full = torch.zeros_like(Kbar)
    fb.focus_pool_keys(ctx, sh, dK, full)
    torch.cuda.synchronize()
    assert torch.equal(Kbar, full)
    touched = sorted({int(p) // B for p in pos if p < s.M})
    untouched = [b for b in range(s.nb) if b not in touched]
    assert torch.equal(Kbar[:, untouched], before[:, untouched]) and not torch.equal(Kbar[:, touched], before[:, touched])
    eK, _ = fo.update_kv(K, V, Kn[:n], Vn[:n], pos)
    ora = fo.pool_keys(wl.storage_to_f64(eK, dtype), s.M, s.B)
    assert np.max(np.abs(Kbar.cpu().numpy().astype(np.float64) - ora)) <= 1e-6 * max(1.0, np.abs(ora).max())
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("dtype,d,H,Hkv", [("bf16", 128, 8, 2), ("f32", 64, 4, 4)])
def test_block_entry_full_refresh(ctx, dtype, d, H, Hkv):
    """The block-entry branch of Algorithm 1 at a small shape: I_active = every position, so all L rows attend densely
    over all L keys (Q holds all L rows, q_base = 0, no row list), every row of the cache is refreshed (Eq. 3 with
    U = everything) and the pooled keys are rebuilt -- each against the oracle."""
    import math
    rng = np.random.default_rng(d + H)
    s = wl.Shape(640, 520, H, Hkv, d, 64, dtype)
    Q = wl.to_storage(rng.standard_normal((s.L, H, d)).astype(np.float32) / math.sqrt(d) * 2, dtype)
    K_old = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    V_old = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    K_new = wl.to_storage(rng.standard_normal((s.L, Hkv, d)).astype(np.float32), dtype)
    V_new = wl.to_storage(rng.standard_normal((s.L, Hkv, d)).astype(np.float32), dtype)
    sh = fstep.c_shape(s)
    dQ, dK, dV = fstep.to_device(Q, dtype), fstep.to_device(K_old, dtype), fstep.to_device(V_old, dtype)
    rows = torch.arange(s.L, dtype=torch.int32, device="cuda")
    n_rows = torch.tensor([s.L], dtype=torch.int32, device="cuda")
    # the layer's new K/V states of all positions replace the cache, then every row attends over the fresh cache
    fb.focus_update_kv(ctx, sh, dK, dV, fstep.to_device(K_new, dtype), fstep.to_device(V_new, dtype), rows, n_rows, s.L)
    O = torch.zeros(s.L, H, d, dtype=fstep.torch_dtype(dtype), device="cuda")
    lse = torch.zeros(H, s.L, dtype=torch.float32, device="cuda")
    fb.focus_dense_attn(ctx, sh, dQ, 0, s.L, None, None, 0, dK, dV, O, lse)
    Kbar = torch.full((Hkv, s.nb, d), 5.0, dtype=torch.float32, device="cuda")
    fb.focus_update_pooled_keys(ctx, sh, dK, Kbar, rows, n_rows, s.L)             # every block holds a refreshed row
    torch.cuda.synchronize()
    eK, eV = fo.update_kv(K_old, V_old, K_new, V_new, range(s.L))
    view = (lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)) if dtype == "bf16" else (lambda t: t.cpu().numpy())
    assert np.array_equal(view(dK), eK) and np.array_equal(view(dV), eV)
    Kf, Vf = wl.storage_to_f64(eK, dtype), wl.storage_to_f64(eV, dtype)
    Od, ld = fo.dense_attn(wl.storage_to_f64(Q, dtype), Kf, Vf, 1.0 / math.sqrt(d))
    tol = 2e-2 if dtype == "bf16" else 1e-5
    assert float(np.max(np.abs(fstep.from_device(O) - Od))) <= tol
    assert float(np.max(np.abs(fstep.from_device(lse) - ld))) <= (2e-3 if dtype == "bf16" else 1e-4)
    ora = fo.pool_keys(Kf, s.M, s.B)
    assert np.max(np.abs(Kbar.cpu().numpy().astype(np.float64) - ora)) <= 1e-6 * max(1.0, np.abs(ora).max())
    assert ctx.poll_status() == 0
