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
