"""GPU parity: every stage of the path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Small shapes span several key tiles, a ragged last prompt block and a ragged response tail."""
import math

import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2602_02159_b200 import binding as fb
from paper_2602_02159_b200 import step as fstep
from paper_2602_02159_b200 import workloads as wl
from tests.helpers import check_topk_band, max_abs, rel_rms

pytestmark = pytest.mark.gpu

TOL_ABS = {"f32": 1e-5, "bf16": 2e-2}       # contractual max-abs on attention outputs
TOL_RMS = {"f32": 1e-5, "bf16": 1e-2}       # self-imposed relative RMS (outputs are ~1e-3..1e-2 in size)
TOL_LSE = {"f32": 1e-4, "bf16": 1e-3}
BAND = 1e-3


@pytest.fixture(scope="module")
def ctx():
    c = fb.Context(0)
    yield c
    assert c.poll_status() == 0
    c.close()


def small_workload(dtype, d, B, H=4, Hkv=4, L=1500, M=1100, k=6, w=8, n_sink=9, C=3, seed=3, blk=None):
    s = wl.Shape(L, M, H, Hkv, d, B, dtype)
    lo, hi = blk if blk else (M, min(L, M + 96))
    return wl.Workload(f"small_{dtype}_{d}_{B}", s, k=k, w=w, n_sink=n_sink, C=C, blk_lo=lo, blk_hi=hi, seed=seed)


SHAPES = [
    pytest.param(("f32", 64, 64, 4, 4), id="f32_d64_B64"),
    pytest.param(("f32", 128, 128, 4, 2), id="f32_d128_gqa"),
    pytest.param(("bf16", 128, 128, 4, 4), id="bf16_d128_B128_mha"),
    pytest.param(("bf16", 128, 128, 8, 2), id="bf16_d128_B128_gqa"),
    pytest.param(("bf16", 64, 64, 4, 4), id="bf16_d64_B64"),
    pytest.param(("bf16", 128, 64, 4, 4), id="bf16_d128_B64"),
]


def make_inputs(w, variant="fix"):
    s = w.shape
    t = wl.gen_qkv(s, w.seed, variant=variant, threads=4)
    c_prev, _ = wl.gen_confidence(w.seed, s.N)
    masked = wl.gen_masked(w)
    rng = np.random.default_rng(w.seed + 100)
    masked[s.M:][rng.random(s.N) < 0.3] = 0            # some gen positions already decoded
    host = dict(Q=wl.storage_to_f64(t["Q"], s.dtype), K=wl.storage_to_f64(t["K"], s.dtype),
                V=wl.storage_to_f64(t["V"], s.dtype), conf=wl.full_conf(s, c_prev), masked=masked,
                sink_pos=t["sink_pos"])
    dev = dict(Q=fstep.to_device(t["Q"], s.dtype), K=fstep.to_device(t["K"], s.dtype),
               V=fstep.to_device(t["V"], s.dtype), conf=torch.from_numpy(host["conf"]).cuda(),
               masked=torch.from_numpy(masked).cuda())
    return host, dev


def oracle_chain(w, host, head_reduce, sink_mode):
    s = w.shape
    scale = 1.0 / math.sqrt(s.d)
    focus, active = fo.select_queries(host["conf"], host["masked"], w.blk_lo, w.blk_hi, w.k, w.w, s.M, s.L)
    Qa = host["Q"][active - s.M]
    S = fo.sink_scores(Qa, host["K"], scale)
    sinks = fo.find_sinks(S, w.n_sink, 0, s.M)
    Kbar = fo.pool_keys(host["K"], s.M, s.B)
    R = fo.score_blocks(host["Q"][focus - s.M], Kbar, head_reduce)
    blocks, keep = fo.select_blocks(R, w.C, sinks, s.B, sink_mode)
    return dict(focus=focus, active=active, S=S, sinks=sinks, Kbar=Kbar, R=R, blocks=blocks, keep=keep, scale=scale)


# --------------------------------------------------------------------------------------------------
def test_select_queries_exact(ctx):
    """Comparison-only stage: bit-exact, no band.  Includes ties, NaN, k > candidates, k = 0, clipping."""
    rng = np.random.default_rng(0)
    cases = []
    for trial in range(12):
        L = int(rng.integers(40, 3000))
        M = int(rng.integers(0, L // 2))
        conf = rng.beta(2, 5, size=L).astype(np.float32)
        if trial % 3 == 0:
            conf = np.round(conf * 8) / 8                     # many ties
        if trial % 4 == 1:
            conf[rng.integers(0, L, size=5)] = np.nan
        if trial % 5 == 2:
            conf[rng.integers(0, L, size=5)] = -0.0
        masked = (rng.random(L) < 0.6).astype(np.uint8)
        lo = int(rng.integers(M, L))
        hi = int(rng.integers(lo, min(L, lo + 600) + 1))
        k = int(rng.integers(0, 40))
        w = int(rng.integers(0, 12))
        cases.append((conf, masked, L, lo, hi, k, w, M, L))
    # the longest decoding block the stage takes (4096 positions), small and large k, ties cut by the threshold, NaNs
    for k_long, quant in ((1, 0), (37, 16), (1024, 64), (600, 4)):
        Lb = 5000
        c = rng.beta(2, 5, size=Lb).astype(np.float32)
        if quant:
            c = np.round(c * quant) / quant
        c[rng.integers(0, Lb, size=9)] = np.nan
        msk = (rng.random(Lb) < 0.7).astype(np.uint8)
        cases.append((c, msk, Lb, 300, 300 + 4096, k_long, 4, 0, Lb))
    cases.append((np.full(5000, 0.25, dtype=np.float32), np.ones(5000, dtype=np.uint8), 5000, 0, 4096, 1000, 2, 0, 5000))
    conf = np.full(64, 0.5, dtype=np.float32)
    cases.append((conf, np.ones(64, dtype=np.uint8), 64, 0, 64, 8, 8, 0, 64))            # all equal
    cases.append((conf, np.zeros(64, dtype=np.uint8), 64, 0, 64, 8, 8, 0, 64))           # nothing masked
    cases.append((conf, np.ones(64, dtype=np.uint8), 64, 10, 10, 8, 8, 0, 64))           # empty block
    cases.append((conf, np.ones(64, dtype=np.uint8), 64, 0, 64, 4, 8, 20, 30))           # clip excludes everything near picks
    for conf, masked, L, lo, hi, k, w, clo, chi in cases:
        span = 2 * (w // 2) + 1
        f = torch.full((max(1, k),), -7, dtype=torch.int32, device="cuda")
        a = torch.full((max(1, k * span),), -7, dtype=torch.int32, device="cuda")
        nf = torch.zeros(1, dtype=torch.int32, device="cuda")
        na = torch.zeros(1, dtype=torch.int32, device="cuda")
        fb.focus_select_queries(ctx, torch.from_numpy(conf).cuda(), torch.from_numpy(masked).cuda(), L, lo, hi, k, w,
                                clo, chi, f, nf, a, na)
        ef, ea = fo.select_queries(conf, masked, lo, hi, k, w, clo, chi)
        assert nf.item() == len(ef) and na.item() == len(ea)
        assert f.cpu().numpy()[:len(ef)].tolist() == ef.tolist()
        assert a.cpu().numpy()[:len(ea)].tolist() == ea.tolist()
        if k > 0:
            assert (f.cpu().numpy()[len(ef):k] == -1).all() and (a.cpu().numpy()[len(ea):k * span] == -1).all()


@pytest.mark.parametrize("cfg", SHAPES)
@pytest.mark.parametrize("force_simt", [False, True], ids=["auto", "simt"])
def test_stages_against_oracle(ctx, cfg, force_simt):
    """Each stage is fed the ORACLE's upstream index sets so that stages are judged in isolation."""
    dtype, d, B, H, Hkv = cfg
    w = small_workload(dtype, d, B, H=H, Hkv=Hkv)
    s = w.shape
    ctx.set_force_simt(force_simt)
    try:
        for head_reduce in (fb.HEADS_PER_KV_GROUP, fb.HEADS_ALL):
            host, dev = make_inputs(w)
            ora = oracle_chain(w, host, head_reduce, fb.SINK_TOKENS)
            b = fstep.StepBuffers(w, head_reduce=head_reduce)
            # stage 1
            fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
            assert b.focus_idx.cpu().numpy()[:b.n_focus.item()].tolist() == ora["focus"].tolist()
            assert b.active_idx.cpu().numpy()[:b.n_active.item()].tolist() == ora["active"].tolist()
            na = len(ora["active"])
            # dense attention over the active rows (+ LSE)
            fstep.dense_layer(ctx, b, dev["Q"], dev["K"], dev["V"])
            Od, lsed = fo.dense_attn(host["Q"][ora["active"] - s.M], host["K"], host["V"], ora["scale"])
            got = fstep.from_device(b.O)[:na]
            assert max_abs(got, Od) <= TOL_ABS[dtype] and rel_rms(got, Od) <= TOL_RMS[dtype]
            assert max_abs(fstep.from_device(b.lse)[:, :na], lsed) <= TOL_LSE[dtype]
            # stage 2, with the dense pass's LSE and with the library computing its own
            for lse_in in (b.lse, None):
                b.sink_idx.fill_(-5)
                fstep.find_sinks(ctx, b, dev["Q"], dev["K"], lse_in)
                S_gpu = fstep.from_device(b.sink_scores)
                assert abs(S_gpu.sum() - 1.0) < 1e-3
                assert np.max(np.abs(S_gpu - ora["S"]) / ora["S"]) < 2e-3
                check_topk_band(b.sink_idx.cpu().numpy(), ora["sinks"], ora["S"], range(0, s.M), BAND, what="sinks")
                assert set(host["sink_pos"].tolist()) <= set(b.sink_idx.cpu().numpy().tolist())
            # stage 3a cold (streams K) and warm (cached K-bar)
            b.sink_idx.copy_(torch.from_numpy(ora["sinks"].astype(np.int32)))
            Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
            fb.focus_pool_keys(ctx, b.shape, dev["K"], Kbar)
            assert max_abs(fstep.from_device(Kbar), ora["Kbar"]) < 1e-5
            for kbar_in in (None, Kbar):
                b.R.zero_()
                fb.focus_score_blocks(ctx, b.shape, dev["Q"], s.M, b.focus_idx, b.n_focus, w.k,
                                      dev["K"] if kbar_in is None else None, kbar_in, head_reduce, b.R)
                Rg = fstep.from_device(b.R).reshape(b.G, s.nb)
                assert max_abs(Rg, ora["R"]) <= 1e-5 * max(1.0, np.abs(ora["R"]).max())
            # stage 3b from the GPU's own scores
            fb.focus_select_blocks(ctx, b.shape, b.R, head_reduce, w.C, b.sink_idx, w.n_sink, fb.SINK_TOKENS,
                                   b.block_idx, b.max_blocks, b.block_cnt, b.sink_keep)
            bi = b.block_idx.cpu().numpy().reshape(b.G, b.max_blocks)
            for g in range(b.G):
                assert b.block_cnt[g].item() == w.C
                check_topk_band(bi[g], ora["blocks"][g], ora["R"][g], range(s.nb), BAND,
                                scale_ref=np.abs(ora["R"][g]).max(), what=f"blocks g{g}")
            # stage 4 on the oracle's sets
            b.block_idx.copy_(torch.from_numpy(np.stack(ora["blocks"]).astype(np.int32).reshape(-1)))
            b.sink_keep.copy_(torch.from_numpy(ora["keep"].reshape(-1)))
            q_rows, n_rows, max_rows = b._rows()
            fb.focus_sparse_attn(ctx, b.shape, dev["Q"], s.M, s.N, q_rows, n_rows, max_rows, dev["K"], dev["V"],
                                 head_reduce, b.block_idx, b.max_blocks, b.block_cnt, b.sink_idx, b.sink_keep,
                                 w.n_sink, b.O, b.lse)
            Os, lses = fo.sparse_attn(host["Q"][ora["active"] - s.M], host["K"], host["V"], s.M, s.B, ora["blocks"],
                                      ora["sinks"], ora["scale"])
            got = fstep.from_device(b.O)[:na]
            assert max_abs(got, Os) <= TOL_ABS[dtype] and rel_rms(got, Os) <= TOL_RMS[dtype]
            assert max_abs(fstep.from_device(b.lse)[:, :na], lses) <= TOL_LSE[dtype]
            assert ctx.poll_status() == 0
    finally:
        ctx.set_force_simt(False)


@pytest.mark.parametrize("cfg", SHAPES)
def test_gen_rows_keep_all_equals_dense_and_sharp_logits(ctx, cfg):
    """All N gen rows as queries (q_rows = NULL); keep ratio 1 must reproduce dense attention; Q, K ~ 1.5 N(0,1)
    gives peaky softmax rows where the 2e-2 bound on bf16 outputs is a meaningful test.  The bounds are the
    contractual ones (2e-2 bf16, 1e-5 fp32, absolute); the values are scaled (0.3 N(0,1)) so that outputs stay below 1
    in magnitude -- an absolute bound of 1e-5 on outputs of size 3 would ask for more than fp32 logits of size 30
    can give (their rounding alone is 30 * 2^-24 = 2e-6 relative in every probability)."""
    dtype, d, B, H, Hkv = cfg
    s = wl.Shape(1400, 1000, H, Hkv, d, B, dtype)
    rng = np.random.default_rng(5)
    Qs = wl.to_storage(rng.standard_normal((s.N, H, d)).astype(np.float32) * 1.5, dtype)
    Ks = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32) * 1.5, dtype)
    Vs = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32) * (1.0 if dtype == "bf16" else 0.3), dtype)
    Q, K, V = (wl.storage_to_f64(x, dtype) for x in (Qs, Ks, Vs))
    dQ, dK, dV = (fstep.to_device(x, dtype) for x in (Qs, Ks, Vs))
    sh = fstep.c_shape(s)
    O = torch.zeros(s.N, H, d, dtype=fstep.torch_dtype(dtype), device="cuda")
    lse = torch.zeros(H, s.N, dtype=torch.float32, device="cuda")
    scale = 1.0 / math.sqrt(d)
    fb.focus_dense_attn(ctx, sh, dQ, s.M, s.N, None, None, 0, dK, dV, O, lse)
    Od, ld = fo.dense_attn(Q, K, V, scale)
    assert np.sqrt(np.mean(Od ** 2)) > (0.05 if dtype == "bf16" else 0.015)
    tol = TOL_ABS[dtype]
    assert max_abs(fstep.from_device(O), Od) <= tol, max_abs(fstep.from_device(O), Od)
    assert max_abs(fstep.from_device(lse), ld) <= (2e-3 if dtype == "bf16" else 1e-4)
    dense_out = O.clone()
    # keep every block, plus sinks that all lie inside kept blocks -> identical key set
    G = Hkv
    nb = s.nb
    bidx = torch.arange(nb, dtype=torch.int32, device="cuda").repeat(G)
    bcnt = torch.full((G,), nb, dtype=torch.int32, device="cuda")
    sinks = torch.tensor([0, 77, 999], dtype=torch.int32, device="cuda")
    keep = torch.zeros(G * 3, dtype=torch.uint8, device="cuda")
    fb.focus_sparse_attn(ctx, sh, dQ, s.M, s.N, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP, bidx, nb, bcnt, sinks,
                         keep, 3, O, lse)
    assert max_abs(fstep.from_device(O), Od) <= tol
    assert max_abs(fstep.from_device(O), fstep.from_device(dense_out)) <= tol
    assert ctx.poll_status() == 0


def test_long_key_pipeline_single_split(ctx):
    """Enough query tiles to fill the GPU (no key split), so each CTA walks all 21 key tiles: the K/V ring
    wraps several times and the running max is rescaled along the way (growing logits)."""
    H, d = 16, 128
    s = wl.Shape(2600, 1300, H, H, d, 128, "bf16")
    rng = np.random.default_rng(11)
    ramp = np.linspace(0.3, 2.0, s.L, dtype=np.float32)[None, :, None]       # later keys score higher
    Qs = wl.to_storage(rng.standard_normal((s.N, H, d)).astype(np.float32), "bf16")
    Ks = wl.to_storage(rng.standard_normal((H, s.L, d)).astype(np.float32) * ramp, "bf16")
    Vs = wl.to_storage(rng.standard_normal((H, s.L, d)).astype(np.float32), "bf16")
    Q, K, V = (wl.storage_to_f64(x, "bf16") for x in (Qs, Ks, Vs))
    dQ, dK, dV = (fstep.to_device(x, "bf16") for x in (Qs, Ks, Vs))
    O = torch.zeros(s.N, H, d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(H, s.N, dtype=torch.float32, device="cuda")
    fb.focus_dense_attn(ctx, fstep.c_shape(s), dQ, s.M, s.N, None, None, 0, dK, dV, O, lse)
    heads = [0, 7, 15]
    Od, ld = fo.dense_attn(Q, K, V, 1.0 / math.sqrt(d), heads=heads)
    got = fstep.from_device(O)
    assert max_abs(got[:, heads], Od[:, heads]) <= 2e-2
    assert max_abs(fstep.from_device(lse)[heads], ld[heads]) <= 2e-3
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("cfg", [SHAPES[0], SHAPES[2], SHAPES[3], SHAPES[5]])
def test_fused_sparse_layer_matches_stagewise_and_oracle(ctx, cfg):
    """focus_sparse_layer (fused selection + attention) against the stage-by-stage calls and the oracle."""
    dtype, d, B, H, Hkv = cfg
    w = small_workload(dtype, d, B, H=H, Hkv=Hkv, n_sink=150, C=4, seed=8)       # two sink tiles
    s = w.shape
    host, dev = make_inputs(w)
    ora = oracle_chain(w, host, fb.HEADS_PER_KV_GROUP, fb.SINK_TOKENS)
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    outs = []
    for fused in (False, True):
        b = fstep.StepBuffers(w)
        fb.focus_pool_keys(ctx, b.shape, dev["K"], Kbar)
        fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
        b.sink_idx.copy_(torch.from_numpy(ora["sinks"].astype(np.int32)))
        fstep.sparse_layer(ctx, b, dev["Q"], dev["K"], dev["V"], Kbar=Kbar, fused=fused)
        torch.cuda.synchronize()
        outs.append(b)
    a, f = outs
    assert torch.equal(a.block_idx, f.block_idx) and torch.equal(a.block_cnt, f.block_cnt)
    assert torch.equal(a.sink_keep, f.sink_keep)
    assert max_abs(fstep.from_device(a.R), fstep.from_device(f.R)) <= 1e-6 * max(1.0, np.abs(ora["R"]).max())
    na = len(ora["active"])
    bi = f.block_idx.cpu().numpy().reshape(s.Hkv, -1)
    for g in range(s.Hkv):
        check_topk_band(bi[g], ora["blocks"][g], ora["R"][g], range(s.nb), BAND, scale_ref=np.abs(ora["R"][g]).max())
    blocks = [bi[g] for g in range(s.Hkv)]
    Os, lses = fo.sparse_attn(host["Q"][ora["active"] - s.M], host["K"], host["V"], s.M, s.B, blocks, ora["sinks"],
                              ora["scale"])
    for b in outs:
        got = fstep.from_device(b.O)[:na]
        assert max_abs(got, Os) <= TOL_ABS[dtype] and rel_rms(got, Os) <= TOL_RMS[dtype]
        assert max_abs(fstep.from_device(b.lse)[:, :na], lses) <= TOL_LSE[dtype]
    assert ctx.poll_status() == 0


def _rand_qkv(s, seed, qk_scale=1.0):
    rng = np.random.default_rng(seed)
    Qs = wl.to_storage(rng.standard_normal((s.N, s.H, s.d)).astype(np.float32) * qk_scale, s.dtype)
    Ks = wl.to_storage(rng.standard_normal((s.Hkv, s.L, s.d)).astype(np.float32) * qk_scale, s.dtype)
    Vs = wl.to_storage(rng.standard_normal((s.Hkv, s.L, s.d)).astype(np.float32), s.dtype)
    return Qs, Ks, Vs


@pytest.mark.parametrize("rows", [40, 128, 512])
@pytest.mark.parametrize("lists", ["even_ragged_second", "odd_ragged_alone", "ragged_first", "single"])
def test_64_token_blocks_are_paired_into_key_tiles(ctx, rows, lists):
    """KV block 64 on the tensor-core path: two selected blocks share one 128-key tile (two 64-row TMA boxes per
    half tile).  Block lists with an even and an odd number of blocks, non-adjacent pairs, the short last block of
    the prompt as the second block of a pair, alone in the last tile, and (list not ascending) as the first of a
    pair; 40 rows take the one-warpgroup kernel, 128 rows the key-pair form, 512 stacked rows per KV head the
    two-tile form or the key-pair form depending on the tile count."""
    M = 64 * 150 + 40                                              # 151 blocks, the last one 40 tokens
    s = wl.Shape(M + rows, M, 4, 4, 128, 64, "bf16") if rows != 512 else wl.Shape(M + 128, M, 8, 2, 128, 64, "bf16")
    nb = s.nb
    assert nb == 151
    rng = np.random.default_rng(11)
    pool = np.sort(rng.choice(nb - 1, size=140, replace=False))
    if lists == "even_ragged_second":
        blocks = [np.concatenate([pool[:69], [nb - 1]]), pool[10:80]]                 # 70 and 70 blocks
    elif lists == "odd_ragged_alone":
        blocks = [np.concatenate([pool[:70], [nb - 1]]), pool[5:76]]                  # 71 and 71 blocks
    elif lists == "ragged_first":
        blocks = [np.concatenate([pool[:68], [nb - 1, pool[100]]]), pool[3:73][::-1].copy()]  # short block, then a full one
    else:
        blocks = [np.array([nb - 1]), np.array([7])]
    blocks = (blocks * s.Hkv)[:s.Hkv]
    C = max(len(b) for b in blocks) + 2
    bidx = np.full((s.Hkv, C), -1, dtype=np.int32)
    for g, b in enumerate(blocks):
        bidx[g, :len(b)] = b
    sinks = np.sort(rng.choice(s.M, size=70, replace=False)).astype(np.int32)
    keep = np.array([[0 if (j // s.B) in set(blocks[g].tolist()) else 1 for j in sinks] for g in range(s.Hkv)],
                    dtype=np.uint8)
    Qs, Ks, Vs = _rand_qkv(s, 41, qk_scale=1.5)
    dQ, dK, dV = (fstep.to_device(x, s.dtype) for x in (Qs, Ks, Vs))
    O = torch.zeros(s.N, s.H, s.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(s.H, s.N, dtype=torch.float32, device="cuda")
    fb.focus_sparse_attn(ctx, fstep.c_shape(s), dQ, s.M, s.N, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP,
                         torch.from_numpy(bidx.reshape(-1)).cuda(), C,
                         torch.tensor([len(b) for b in blocks], dtype=torch.int32, device="cuda"),
                         torch.from_numpy(sinks).cuda(), torch.from_numpy(keep.reshape(-1)).cuda(), len(sinks), O, lse)
    assert ctx.last_attn_variant() in (2, 3, 4)
    hpg = s.H // s.Hkv
    scale = 1.0 / math.sqrt(s.d)
    f64h = lambda a, h, kv=True: wl.storage_to_f64(a[h // hpg:h // hpg + 1] if kv else a[:, h:h + 1], s.dtype)
    got, got_lse = fstep.from_device(O), fstep.from_device(lse)
    for h in (0, s.H - 1):
        Oh, lh = fo.sparse_attn(f64h(Qs, h, False), f64h(Ks, h), f64h(Vs, h), s.M, s.B, [blocks[h // hpg]], sinks, scale)
        assert max_abs(got[:, h], Oh[:, 0]) <= 2e-2 and rel_rms(got[:, h], Oh[:, 0]) <= 1e-2
        assert max_abs(got_lse[h], lh[0]) <= 2e-3
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("merge", ["cluster", "counters", "kernel"])
@pytest.mark.parametrize("rows", [40, 128, 512])
@pytest.mark.parametrize("keys", ["dense", "sparse_B64", "sparse_B128"])
def test_head_dim_64_runs_on_the_tensor_core_kernels(keys, rows, merge):
    """bf16 with head dim 64 (Dream-style heads are 128 wide, smaller models 64): the tensor-core kernels keep their
    128-wide geometry and receive the missing upper half of every K/V tile as zeros (a copy that lies wholly outside
    the tensor), the upper half of the query tile is staged as zeros, and only 64 output columns are written.  All
    three kernel forms (40 / 128 / 512 stacked rows per KV head), dense and sparse key sets with both block sizes,
    sink tiles, a ragged last block, key splits merged in all three ways, row lists, lse -- against the oracle; the
    output buffer is twice as long as needed and its tail must stay untouched."""
    if merge != "cluster" and rows != 40:
        pytest.skip("only the one-tile kernel merges through global memory")
    B = 64 if keys == "sparse_B64" else 128
    # 512 stacked rows: GQA 4:1 with 128 rows; the dense case has enough KV heads and keys for the two-tile form
    wide = rows == 512 and keys == "dense"
    M = 64 * (200 if wide else 150) + 40
    H, Hkv = ((64, 16) if wide else (8, 2)) if rows == 512 else (4, 4)
    n = 128 if rows == 512 else rows
    s = wl.Shape(M + n, M, H, Hkv, 64, B, "bf16")
    rng = np.random.default_rng(5)
    Qs, Ks, Vs = _rand_qkv(s, 61, qk_scale=1.5)
    dQ, dK, dV = (fstep.to_device(x, s.dtype) for x in (Qs, Ks, Vs))
    # a row list: every row but three, in order
    q_rows = np.array([r for r in range(n) if r not in (3, 17, n - 1)], dtype=np.int32) + M
    n_rows = len(q_rows)
    d_rows = torch.from_numpy(np.concatenate([q_rows, np.full(3, -1, np.int32)])).cuda()
    d_nrows = torch.tensor([n_rows], dtype=torch.int32, device="cuda")
    O = torch.full((2 * n, s.H, s.d), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(s.H, n, dtype=torch.float32, device="cuda")
    c = fb.Context(0, workspace_bytes=64 << 20)
    try:
        if merge != "cluster":
            c.set_option(fb.OPT_MERGE_MODE, fb.MERGE_COUNTERS if merge == "counters" else fb.MERGE_KERNEL)
        sh = fstep.c_shape(s)
        if keys == "dense":
            fb.focus_dense_attn(c, sh, dQ, s.M, n, d_rows, d_nrows, n, dK, dV, O, lse)
        else:
            nb = s.nb
            blocks = [np.sort(np.concatenate([rng.choice(nb - 1, size=(100 if B == 64 else 50) + g, replace=False), [nb - 1]])) for g in range(Hkv)]
            C = max(len(b) for b in blocks) + 1
            bidx = np.full((Hkv, C), -1, dtype=np.int32)
            for g, b in enumerate(blocks):
                bidx[g, :len(b)] = b
            sinks = np.sort(rng.choice(s.M, size=70, replace=False)).astype(np.int32)
            keep = np.array([[0 if (j // B) in set(blocks[g].tolist()) else 1 for j in sinks] for g in range(Hkv)],
                            dtype=np.uint8)
            fb.focus_sparse_attn(c, sh, dQ, s.M, n, d_rows, d_nrows, n, dK, dV, fb.HEADS_PER_KV_GROUP,
                                 torch.from_numpy(bidx.reshape(-1)).cuda(), C,
                                 torch.tensor([len(b) for b in blocks], dtype=torch.int32, device="cuda"),
                                 torch.from_numpy(sinks).cuda(), torch.from_numpy(keep.reshape(-1)).cuda(), len(sinks),
                                 O, lse)
        torch.cuda.synchronize()
        assert c.last_attn_variant() == (3 if wide else {40: 2, 128: 4, 512: 4}[rows])
        assert c.poll_status() == 0
    finally:
        c.close()
    assert bool((O[n_rows:].float() == 7.0).all()), "rows past the row count (and the spare half) stay untouched"
    hpg = s.H // s.Hkv
    scale = 1.0 / math.sqrt(s.d)
    f64h = lambda a, h, kv=True: wl.storage_to_f64(a[h // hpg:h // hpg + 1] if kv else a[:, h:h + 1], s.dtype)
    got, got_lse = fstep.from_device(O)[:n_rows], fstep.from_device(lse)[:, :n_rows]
    for h in (0, s.H - 1):
        Qh = f64h(Qs, h, False)[q_rows - M]
        if keys == "dense":
            Oh, lh = fo.dense_attn(Qh, f64h(Ks, h), f64h(Vs, h), scale)
        else:
            Oh, lh = fo.sparse_attn(Qh, f64h(Ks, h), f64h(Vs, h), s.M, s.B, [blocks[h // hpg]], sinks, scale)
        assert max_abs(got[:, h], Oh[:, 0]) <= 2e-2 and rel_rms(got[:, h], Oh[:, 0]) <= 1e-2
        assert max_abs(got_lse[h], lh[0]) <= 2e-3


@pytest.mark.parametrize("world", [2, 4])
@pytest.mark.parametrize("cfg", [("bf16", 128, 128, 8, 4), ("f32", 64, 64, 8, 8)])
def test_sinks_of_a_layer_whose_heads_are_dealt_out_to_several_ranks(ctx, cfg, world):
    """Eq. 6 is a mean over all heads: the one step of the path that needs an exchange when the heads of a layer
    live on several GPUs.  Here the ranks run one after the other on one GPU -- every rank computes S over its own
    heads (focus_find_sinks with n_sink = 0), the mean over ranks stands in for the all-reduce, focus_select_sinks
    takes the Top-N_sink -- and the result is held against the oracle over all heads (band rule), against the
    single-device call, and against an exact selection on the averaged float32 scores themselves."""
    from paper_2602_02159_b200 import head_shards
    dtype, d, B, H, Hkv = cfg
    w = small_workload(dtype, d, B, H=H, Hkv=Hkv, L=2600, M=2100, n_sink=21)
    s = w.shape
    host, dev = make_inputs(w)
    b = fstep.StepBuffers(w)
    fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
    fstep.find_sinks(ctx, b, dev["Q"], dev["K"], None)
    single = b.sink_idx.cpu().numpy().copy()
    S_single = fstep.from_device(b.sink_scores).copy()
    S_sum = torch.zeros(s.L, dtype=torch.float32, device="cuda")
    for r in range(world):
        qh, kvh = head_shards.local_heads(H, Hkv, r, world)
        shape_r = fb.make_shape(s.L, s.M, H // world, Hkv // world, d, B, fb.F32 if dtype == "f32" else fb.BF16,
                                q_stride_row=H * d, q_stride_head=d, kv_stride_tok=d, kv_stride_head=s.L * d)
        S_r = torch.full((s.L,), 9.0, dtype=torch.float32, device="cuda")
        fb.focus_find_sinks(ctx, shape_r, dev["Q"][:, qh], s.M, b.active_idx, b.n_active, b.max_active, dev["K"][kvh],
                            None, 0, 0, s.M, None, S_r)
        S_sum += S_r
    S_mean = (S_sum * (1.0 / world)).contiguous()
    sink = torch.full((w.n_sink,), -7, dtype=torch.int32, device="cuda")
    fb.focus_select_sinks(ctx, S_mean, s.L, 0, s.M, w.n_sink, sink)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got, S_got = sink.cpu().numpy(), fstep.from_device(S_mean)
    na = int(b.n_active.item())
    active = b.active_idx.cpu().numpy()[:na]
    S_ora = fo.sink_scores(host["Q"][active - s.M], host["K"], 1.0 / math.sqrt(d))
    ora = fo.find_sinks(S_ora, w.n_sink, 0, s.M)
    assert np.max(np.abs(S_got - S_ora) / S_ora) < 2e-3                     # the bar of the single-device scores
    assert max_abs(S_got, S_single) <= 1e-6 * float(S_ora.max())          # same scores up to the order of the head sum
    check_topk_band(got, ora, S_ora, range(s.M), BAND, what=f"sharded sinks, {world} ranks")
    check_topk_band(got, [int(i) for i in single if i >= 0], S_single.astype(np.float64), range(s.M), BAND,
                    what="sharded against single device")
    assert got.tolist() == fo.find_sinks(S_got.astype(np.float64), w.n_sink, 0, s.M).tolist(), "exact on its own scores"


def test_a_rank_of_a_head_sharded_layer_computes_what_the_single_device_computes_for_its_heads(ctx):
    """Two ranks, one after the other on one GPU, each with its half of the KV heads (views into the full tensors by
    strides): dense layer, sink scores over the own heads, the mean over ranks (a sum here), Top-N_sink, sparse
    layer.  Given the same sink set, everything else is per KV group: the rank's block lists and keep flags must be
    exactly those of the single-device run for its groups, its attention outputs those of the single-device run for
    its heads (to rounding: fewer heads per launch means other key splits, i.e. another summation order)."""
    import dataclasses
    from paper_2602_02159_b200 import head_shards
    world = 2
    w = small_workload("bf16", 128, 128, H=8, Hkv=4, L=2600, M=2100, n_sink=21, C=5)
    s = w.shape
    host, dev = make_inputs(w)
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    fb.focus_pool_keys(ctx, fstep.c_shape(s), dev["K"], Kbar)
    ranks = []
    S_sum = torch.zeros(s.L, dtype=torch.float32, device="cuda")
    for r in range(world):
        qh, kvh = head_shards.local_heads(s.H, s.Hkv, r, world)
        w_r = dataclasses.replace(w, shape=wl.Shape(s.L, s.M, s.H // world, s.Hkv // world, s.d, s.B, s.dtype))
        b = fstep.StepBuffers(w_r)
        b.shape = fb.make_shape(s.L, s.M, s.H // world, s.Hkv // world, s.d, s.B, fb.BF16, q_stride_row=s.H * s.d,
                                q_stride_head=s.d, kv_stride_tok=s.d, kv_stride_head=s.L * s.d)
        Q, K, V = dev["Q"][:, qh], dev["K"][kvh], dev["V"][kvh]
        fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
        fstep.dense_layer(ctx, b, Q, K, V)
        dense = b.O.clone()
        fstep.find_sinks_sharded(ctx, b, Q, K, b.lse)          # no process group: the local scores stay in b.sink_scores
        S_sum += b.sink_scores
        ranks.append(dict(b=b, Q=Q, K=K, V=V, qh=qh, kvh=kvh, dense=dense))
    S_mean = (S_sum * (1.0 / world)).contiguous()
    for rk in ranks:                                           # what the all-reduce leaves on every rank
        rk["b"].sink_scores.copy_(S_mean)
        fb.focus_select_sinks(ctx, rk["b"].sink_scores, s.L, 0, s.M, w.n_sink, rk["b"].sink_idx)
        fstep.sparse_layer(ctx, rk["b"], rk["Q"], rk["K"], rk["V"], Kbar=Kbar[rk["kvh"]].contiguous())
    assert torch.equal(ranks[0]["b"].sink_idx, ranks[1]["b"].sink_idx)
    # the single device, with the same sink set
    b1 = fstep.StepBuffers(w)
    fstep.select_queries(ctx, b1, dev["conf"], dev["masked"])
    fstep.dense_layer(ctx, b1, dev["Q"], dev["K"], dev["V"])
    dense1 = b1.O.clone()
    fstep.find_sinks(ctx, b1, dev["Q"], dev["K"], b1.lse)
    assert float((b1.sink_scores - S_mean).abs().max()) <= 1e-6 * float(S_mean.max())
    b1.sink_idx.copy_(ranks[0]["b"].sink_idx)
    fstep.sparse_layer(ctx, b1, dev["Q"], dev["K"], dev["V"], Kbar=Kbar)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    na = int(b1.n_active.item())
    per = s.Hkv // world
    for r, rk in enumerate(ranks):
        b = rk["b"]
        assert torch.equal(b.active_idx, b1.active_idx) and torch.equal(b.focus_idx, b1.focus_idx)
        assert torch.equal(b.block_cnt, b1.block_cnt[r * per:(r + 1) * per])
        assert torch.equal(b.block_idx.view(per, -1), b1.block_idx.view(s.Hkv, -1)[r * per:(r + 1) * per])
        assert torch.equal(b.sink_keep.view(per, -1), b1.sink_keep.view(s.Hkv, -1)[r * per:(r + 1) * per])
        assert torch.equal(b.R.view(per, -1), b1.R.view(s.Hkv, -1)[r * per:(r + 1) * per])
        for mine, ref in ((rk["dense"], dense1), (b.O, b1.O)):
            a, c = fstep.from_device(mine)[:na], fstep.from_device(ref)[:na, rk["qh"]]
            assert max_abs(a, c) <= 2e-2 and rel_rms(a, c) <= 5e-3


@pytest.mark.parametrize("heads", [1, 74])
@pytest.mark.parametrize("tiles", [1, 2, 3, 4, 5, 7, 8, 10, 12, 21, 24, 26])
def test_one_tile_kernel_with_every_short_key_loop(ctx, heads, tiles):
    """The one-tile kernel's K/V ring has three or four slots in use depending on the key tiles per CTA (cross-over at
    12), requests three copies at the start and the rest once the first has landed, and its P V products commit to two
    barriers by tile parity: dense attention with key loops of 1 to 13 tiles per CTA, odd and even, a ragged last
    tile, with one head (many splits of few tiles) and with 74 heads (two splits: tiles / 2 per CTA)."""
    L = tiles * 128 - 37
    n = 24
    s = wl.Shape(L, L - n, heads, heads, 128, 128, "bf16")
    Qs, Ks, Vs = _rand_qkv(s, 100 + tiles, qk_scale=1.5)
    dQ, dK, dV = (fstep.to_device(x, s.dtype) for x in (Qs, Ks, Vs))
    O = torch.zeros(n, s.H, s.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(s.H, n, dtype=torch.float32, device="cuda")
    fb.focus_dense_attn(ctx, fstep.c_shape(s), dQ, s.M, n, None, None, 0, dK, dV, O, lse)
    torch.cuda.synchronize()
    assert ctx.last_attn_variant() == 2 and ctx.poll_status() == 0
    got, got_lse = fstep.from_device(O), fstep.from_device(lse)
    f64h = lambda a, h, kv=True: wl.storage_to_f64(a[h:h + 1] if kv else a[:, h:h + 1], s.dtype)
    for h in sorted({0, heads - 1}):
        Oh, lh = fo.dense_attn(f64h(Qs, h, False), f64h(Ks, h), f64h(Vs, h), 1.0 / math.sqrt(s.d))
        assert max_abs(got[:, h], Oh[:, 0]) <= 2e-2 and rel_rms(got[:, h], Oh[:, 0]) <= 1e-2, (tiles, h)
        assert max_abs(got_lse[h], lh[0]) <= 2e-3, (tiles, h)


@pytest.mark.parametrize("cfg", [SHAPES[0], SHAPES[3], SHAPES[5]])
def test_token_major_cache_and_padded_query_rows(ctx, cfg):
    """Strides are part of the shape: K/V cache stored token-major ([L, Hkv, d]: token stride Hkv*d, head stride d)
    and Q rows padded (row stride H*d + 64).  Every stage must give bit for bit what it gives on the contiguous
    layout (same arithmetic, other addresses), which the other tests tie to the oracle; the sparse-layer output is
    also checked against the oracle directly."""
    dtype, d, B, H, Hkv = cfg
    w = small_workload(dtype, d, B, H=H, Hkv=Hkv, n_sink=150, C=4, seed=9)
    s = w.shape
    host, dev = make_inputs(w)
    ora = oracle_chain(w, host, fb.HEADS_PER_KV_GROUP, fb.SINK_TOKENS)
    Kt = dev["K"].permute(1, 0, 2).contiguous()                    # [L, Hkv, d]
    Vt = dev["V"].permute(1, 0, 2).contiguous()
    Qp = torch.zeros(s.N, H * d + 64, dtype=dev["Q"].dtype, device="cuda")
    Qp[:, :H * d] = dev["Q"].reshape(s.N, H * d)
    strided = fb.make_shape(s.L, s.M, H, Hkv, d, B, fb.F32 if dtype == "f32" else fb.BF16,
                            q_stride_row=H * d + 64, q_stride_head=d, kv_stride_tok=Hkv * d, kv_stride_head=d)
    rng = np.random.default_rng(3)
    results = []
    for layout in ("contiguous", "strided"):
        Q, K, V = (dev["Q"], dev["K"], dev["V"]) if layout == "contiguous" else (Qp, Kt, Vt)
        b = fstep.StepBuffers(w)
        if layout == "strided":
            b.shape = strided
        fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
        fstep.dense_layer(ctx, b, Q, K, V)
        dense = (b.O.clone(), b.lse.clone())
        fstep.find_sinks(ctx, b, Q, K, b.lse)
        Kbar = torch.zeros(Hkv, s.nb, d, dtype=torch.float32, device="cuda")
        fb.focus_pool_keys(ctx, b.shape, K, Kbar)
        fb.focus_score_blocks(ctx, b.shape, Q, s.M, b.focus_idx, b.n_focus, max(1, w.k), K, None, fb.HEADS_PER_KV_GROUP, b.R)
        R_cold = b.R.clone()
        outs = []
        for fused in (False, True):
            fstep.sparse_layer(ctx, b, Q, K, V, Kbar=Kbar, fused=fused)
            outs.append((b.O.clone(), b.lse.clone(), b.block_idx.clone(), b.sink_keep.clone(), b.R.clone()))
        # Eq. 3 refresh of the active rows in the layout at hand
        na = b.n_active.item()
        Kn = torch.from_numpy(rng.standard_normal((b.max_active, Hkv, d)).astype(np.float32)).cuda().to(K.dtype)
        Kc, Vc = K.clone(), V.clone()
        fb.focus_update_kv(ctx, b.shape, Kc, Vc, Kn, Kn, b.active_idx, b.n_active, b.max_active)
        if layout == "strided":
            Kc, Vc = Kc.permute(1, 0, 2).contiguous(), Vc.permute(1, 0, 2).contiguous()
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        results.append(dict(dense=dense, sinks=b.sink_idx.clone(), scores=b.sink_scores.clone(), Kbar=Kbar, R_cold=R_cold,
                            outs=outs, Kc=Kc, Vc=Vc, na=na, active=b.active_idx.clone()))
        rng = np.random.default_rng(3)                              # the same new rows for the second layout
    a, z = results
    assert torch.equal(a["active"], z["active"]) and torch.equal(a["sinks"], z["sinks"])
    for x, y in zip(a["dense"], z["dense"]):
        assert torch.equal(x, y)
    assert torch.equal(a["scores"], z["scores"]) and torch.equal(a["Kbar"], z["Kbar"]) and torch.equal(a["R_cold"], z["R_cold"])
    for oa, oz in zip(a["outs"], z["outs"]):
        for x, y in zip(oa, oz):
            assert torch.equal(x, y)
    assert torch.equal(a["Kc"], z["Kc"]) and torch.equal(a["Vc"], z["Vc"])
    # and the strided sparse layer against the oracle
    na = z["na"]
    bi = z["outs"][1][2].cpu().numpy().reshape(Hkv, -1)
    blocks = [bi[g][bi[g] >= 0] for g in range(Hkv)]
    Os, lses = fo.sparse_attn(host["Q"][ora["active"] - s.M], host["K"], host["V"], s.M, s.B, blocks,
                              z["sinks"].cpu().numpy(), ora["scale"])
    got = fstep.from_device(z["outs"][1][0])[:na]
    assert max_abs(got, Os) <= TOL_ABS[dtype] and rel_rms(got, Os) <= TOL_RMS[dtype]
    assert max_abs(fstep.from_device(z["outs"][1][1])[:, :na], lses) <= TOL_LSE[dtype]


@pytest.mark.parametrize("B", [128, 64])
def test_bad_block_index_on_the_tensor_core_path_is_reported_not_dereferenced(ctx, B):
    """An out-of-range or negative entry inside the counted part of a block list masks its key tile (with 64-token
    blocks: the pair it belongs to) and raises INVALID_ARG in the status word; the output stays finite and the
    context usable."""
    s = wl.Shape(6000 + 40, 6000, 4, 4, 128, B, "bf16")
    rng = np.random.default_rng(17)
    good = np.sort(rng.choice(s.nb, size=9, replace=False)).astype(np.int32)
    Qs, Ks, Vs = _rand_qkv(s, 47)
    dQ, dK, dV = (fstep.to_device(x, s.dtype) for x in (Qs, Ks, Vs))
    sinks = np.sort(rng.choice(s.M, size=20, replace=False)).astype(np.int32)
    for bad in (10 ** 6, -5):
        lst = good.copy()
        lst[4] = bad
        bidx = np.tile(lst, (s.Hkv, 1))
        keep = np.ones((s.Hkv, len(sinks)), dtype=np.uint8)
        O = torch.full((s.N, s.H, s.d), 7.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(s.H, s.N, dtype=torch.float32, device="cuda")
        fb.focus_sparse_attn(ctx, fstep.c_shape(s), dQ, s.M, s.N, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP,
                             torch.from_numpy(bidx.reshape(-1)).cuda(), len(lst),
                             torch.full((s.Hkv,), len(lst), dtype=torch.int32, device="cuda"),
                             torch.from_numpy(sinks).cuda(), torch.from_numpy(keep.reshape(-1)).cuda(), len(sinks), O, lse)
        assert ctx.last_attn_variant() == 2
        assert ctx.poll_status() == fb.ERR_INVALID_ARG
        assert torch.isfinite(O.float()).all() and torch.isfinite(lse).all()
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("rows", [40, 128, 256])
@pytest.mark.parametrize("B", [128, 64])
def test_block_lists_too_long_to_stage_in_shared_memory(ctx, B, rows):
    """A split with more key tiles than the shared-memory tile list holds (128, or 96 in the three-warpgroup
    kernels) derives every tile from the block list in global memory instead.  One head, every block of a 140K-token
    prompt but a few selected: ~137 key tiles for each of the 8 splits, with both block sizes (64-token blocks are
    paired) and all three kernel forms (40, 128, 256 rows)."""
    nblk128 = 1100
    M = 128 * nblk128 + 50                                         # the last block is short
    s = wl.Shape(M + rows, M, 1, 1, 128, B, "bf16")
    nb = s.nb
    rng = np.random.default_rng(13)
    drop = set(rng.choice(nb - 1, size=7, replace=False).tolist())
    blocks = [np.array([b for b in range(nb) if b not in drop])]
    C = nb
    bidx = np.full((1, C), -1, dtype=np.int32)
    bidx[0, :len(blocks[0])] = blocks[0]
    sinks = np.sort(rng.choice(s.M, size=40, replace=False)).astype(np.int32)
    keep = np.array([[0 if (j // s.B) in set(blocks[0].tolist()) else 1 for j in sinks]], dtype=np.uint8)
    Qs, Ks, Vs = _rand_qkv(s, 43, qk_scale=1.5)
    dQ, dK, dV = (fstep.to_device(x, s.dtype) for x in (Qs, Ks, Vs))
    O = torch.zeros(s.N, s.H, s.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(s.H, s.N, dtype=torch.float32, device="cuda")
    big = fb.Context(0, workspace_bytes=64 << 20)
    try:
        fb.focus_sparse_attn(big, fstep.c_shape(s), dQ, s.M, s.N, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP,
                             torch.from_numpy(bidx.reshape(-1)).cuda(), C,
                             torch.tensor([len(blocks[0])], dtype=torch.int32, device="cuda"),
                             torch.from_numpy(sinks).cuda(), torch.from_numpy(keep.reshape(-1)).cuda(), len(sinks), O, lse)
        assert big.last_attn_variant() == {40: 2, 128: 4, 256: 3}[rows]
        assert big.poll_status() == 0
    finally:
        big.close()
    f64 = lambda a: wl.storage_to_f64(a, s.dtype)
    Oh, lh = fo.sparse_attn(f64(Qs), f64(Ks), f64(Vs), s.M, s.B, blocks, sinks, 1.0 / math.sqrt(s.d))
    got, got_lse = fstep.from_device(O), fstep.from_device(lse)
    assert max_abs(got[:, 0], Oh[:, 0]) <= 2e-2 and rel_rms(got[:, 0], Oh[:, 0]) <= 1e-2
    assert max_abs(got_lse[0], lh[0]) <= 2e-3


@pytest.mark.parametrize("case", ["dense_split8", "dense_nosplit", "sparse_gqa_split8", "sparse_few_tiles"])
def test_key_pair_kernel(ctx, case):
    """Shapes that take the key-pair attention kernel (one 128-row query tile, two softmax warpgroups on alternating
    key tiles, halves merged in the epilogue): at least 128 stacked rows per KV head, too few key tiles per CTA for
    the two-query-tile kernel.  Covers the cluster merge of 8 splits with odd and even tile counts per split, the
    unsplit case with a ragged last query tile, GQA row stacking, sparse tile lists with sink tiles and a ragged
    last block, splits that end up with one key tile or none (one warpgroup idle / empty partial), and running-max
    rescales (logit std ~1)."""
    if case == "dense_split8":
        s = wl.Shape(9000, 8872, 8, 8, 128, 128, "bf16")            # 128 rows/head, 71 key tiles, 8 CTAs x 8 splits
        heads = [0, 5]
    elif case == "dense_nosplit":
        s = wl.Shape(2500, 1900, 32, 32, 128, 128, "bf16")          # 600 rows/head -> 160 CTAs, 20 tiles each
        heads = [0, 31]
    else:
        s = wl.Shape(20000, 19872, 8, 2, 128, 128, "bf16")          # GQA 4:1 -> 512 stacked rows per KV head
        heads = [1, 6]
    Qs, Ks, Vs = _rand_qkv(s, 37, qk_scale=1.5)
    dQ, dK, dV = (fstep.to_device(x, s.dtype) for x in (Qs, Ks, Vs))
    sh = fstep.c_shape(s)
    O = torch.zeros(s.N, s.H, s.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(s.H, s.N, dtype=torch.float32, device="cuda")
    scale = 1.0 / math.sqrt(s.d)
    hpg = s.H // s.Hkv
    f64h = lambda a, h, kv=True: wl.storage_to_f64(a[h // hpg:h // hpg + 1] if kv else a[:, h:h + 1], s.dtype)
    if case.startswith("dense"):
        fb.focus_dense_attn(ctx, sh, dQ, s.M, s.N, None, None, 0, dK, dV, O, lse)
        ref = {h: fo.dense_attn(f64h(Qs, h, False), f64h(Ks, h), f64h(Vs, h), scale) for h in heads}
    else:
        nb = s.nb                                                  # 156 blocks, the last one short (32 tokens)
        rng = np.random.default_rng(7)
        few = case == "sparse_few_tiles"
        # 40 (39) blocks + 3 sink tiles + 1 response tile over 8 splits: five or six tiles per split;
        # "few": room for 40 blocks but 2 and 1 selected -> 5 or 6 tiles in all, some splits get one tile or none
        blocks = [np.sort(rng.choice(nb, size=n, replace=False)) for n in ((2, 1) if few else (40, 39))]
        blocks[0][-1] = nb - 1                                     # make sure the ragged block is in one list
        blocks[0] = np.unique(blocks[0])
        C = 40
        bidx = np.full((s.Hkv, C), -1, dtype=np.int32)
        for g, b in enumerate(blocks):
            bidx[g, :len(b)] = b
        sinks = np.sort(rng.choice(s.M, size=300, replace=False)).astype(np.int32)
        keep = np.array([[0 if (j // s.B) in set(blocks[g].tolist()) else 1 for j in sinks] for g in range(s.Hkv)],
                        dtype=np.uint8)
        fb.focus_sparse_attn(ctx, sh, dQ, s.M, s.N, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP,
                             torch.from_numpy(bidx.reshape(-1)).cuda(), C,
                             torch.tensor([len(b) for b in blocks], dtype=torch.int32, device="cuda"),
                             torch.from_numpy(sinks).cuda(), torch.from_numpy(keep.reshape(-1)).cuda(), len(sinks), O, lse)
        ref = {h: fo.sparse_attn(f64h(Qs, h, False), f64h(Ks, h), f64h(Vs, h), s.M, s.B, [blocks[h // hpg]], sinks, scale)
               for h in heads}
    assert ctx.last_attn_variant() == 4, "the shape was meant to take the key-pair kernel"
    got, got_lse = fstep.from_device(O), fstep.from_device(lse)
    for h in heads:
        Oh, lh = ref[h]
        assert np.sqrt(np.mean(Oh ** 2)) > 0.02
        assert max_abs(got[:, h], Oh[:, 0]) <= 2e-2 and rel_rms(got[:, h], Oh[:, 0]) <= 1e-2
        assert max_abs(got_lse[h], lh[0]) <= 2e-3
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("case", ["dense_split8", "dense_nosplit", "sparse_gqa_split8"])
def test_two_query_tile_kernel(ctx, case):
    """Shapes that take the 256-row (two query tiles per CTA) attention kernel: >= 256 stacked rows per KV head and
    >= 24 key tiles per CTA (here 32 and more).  Covers the cluster merge of 8 splits, the unsplit case, GQA row stacking, sparse tile
    lists with sink tiles and a ragged last block, and running-max rescales (logit std ~1)."""
    if case == "dense_split8":
        s = wl.Shape(33000, 32744, 8, 8, 128, 128, "bf16")          # 256 rows/head, 258 key tiles, 8 CTAs x 8 splits
        heads = [0, 5]
    elif case == "dense_nosplit":
        s = wl.Shape(5600, 4320, 32, 32, 128, 128, "bf16")          # 1280 rows/head -> 160 CTAs, 44 tiles each
        heads = [0, 31]
    else:
        s = wl.Shape(34000, 33872, 8, 2, 128, 128, "bf16")          # GQA 4:1 -> 512 stacked rows per KV head
        heads = [1, 6]
    Qs, Ks, Vs = _rand_qkv(s, 31, qk_scale=1.5)
    dQ, dK, dV = (fstep.to_device(x, s.dtype) for x in (Qs, Ks, Vs))
    sh = fstep.c_shape(s)
    O = torch.zeros(s.N, s.H, s.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(s.H, s.N, dtype=torch.float32, device="cuda")
    scale = 1.0 / math.sqrt(s.d)
    hpg = s.H // s.Hkv
    f64h = lambda a, h, kv=True: wl.storage_to_f64(a[h // hpg:h // hpg + 1] if kv else a[:, h:h + 1], s.dtype)
    if case.startswith("dense"):
        fb.focus_dense_attn(ctx, sh, dQ, s.M, s.N, None, None, 0, dK, dV, O, lse)
        ref = {h: fo.dense_attn(f64h(Qs, h, False), f64h(Ks, h), f64h(Vs, h), scale) for h in heads}
    else:
        nb = s.nb                                                  # 265 blocks, the last one short (80 tokens)
        rng = np.random.default_rng(5)
        blocks = [np.sort(rng.choice(nb, size=258, replace=False)) for _ in range(s.Hkv)]
        blocks[0][-1] = nb - 1                                     # make sure the ragged block is in one list
        blocks[0] = np.unique(blocks[0])
        C = max(len(b) for b in blocks)
        bidx = np.full((s.Hkv, C), -1, dtype=np.int32)
        for g, b in enumerate(blocks):
            bidx[g, :len(b)] = b
        sinks = np.sort(rng.choice(s.M, size=300, replace=False)).astype(np.int32)
        keep = np.array([[0 if (j // s.B) in set(blocks[g].tolist()) else 1 for j in sinks] for g in range(s.Hkv)],
                        dtype=np.uint8)
        fb.focus_sparse_attn(ctx, sh, dQ, s.M, s.N, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP,
                             torch.from_numpy(bidx.reshape(-1)).cuda(), C,
                             torch.tensor([len(b) for b in blocks], dtype=torch.int32, device="cuda"),
                             torch.from_numpy(sinks).cuda(), torch.from_numpy(keep.reshape(-1)).cuda(), len(sinks), O, lse)
        ref = {h: fo.sparse_attn(f64h(Qs, h, False), f64h(Ks, h), f64h(Vs, h), s.M, s.B, [blocks[h // hpg]], sinks, scale)
               for h in heads}
    assert ctx.last_attn_variant() == 3, "the shape was meant to take the two-query-tile kernel"
    got, got_lse = fstep.from_device(O), fstep.from_device(lse)
    for h in heads:
        Oh, lh = ref[h]
        assert np.sqrt(np.mean(Oh ** 2)) > 0.02
        assert max_abs(got[:, h], Oh[:, 0]) <= 2e-2 and rel_rms(got[:, h], Oh[:, 0]) <= 1e-2
        assert max_abs(got_lse[h], lh[0]) <= 2e-3
    assert ctx.poll_status() == 0


def test_degenerate_cases(ctx):
    """C = 0 with no sinks (response keys only), n_sink = 0, Q = 0 (uniform weights pin the key set),
    a single query row, block list given in descending order."""
    dtype, d, B, H, Hkv = "bf16", 128, 128, 4, 2
    s = wl.Shape(900, 700, H, Hkv, d, B, dtype)          # nb = 6, last block 60 tokens; response 200 (ragged)
    rng = np.random.default_rng(9)
    Ks = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    Vs = wl.to_storage(rng.standard_normal((Hkv, s.L, d)).astype(np.float32), dtype)
    K, V = wl.storage_to_f64(Ks, dtype), wl.storage_to_f64(Vs, dtype)
    dK, dV = fstep.to_device(Ks, dtype), fstep.to_device(Vs, dtype)
    sh = fstep.c_shape(s)
    for force in (False, True):
        ctx.set_force_simt(force)
        for nrow in (1, 200):
            Qz = torch.zeros(s.N, H, d, dtype=torch.bfloat16, device="cuda")
            O = torch.zeros(nrow, H, d, dtype=torch.bfloat16, device="cuda")
            lse = torch.zeros(H, nrow, dtype=torch.float32, device="cuda")
            blocks = [np.array([5, 2]), np.array([0])]
            bidx = torch.tensor([5, 2, 0, -1], dtype=torch.int32, device="cuda")
            bcnt = torch.tensor([2, 1], dtype=torch.int32, device="cuda")
            sinks_np = np.array([3, 300, 650])                                  # 300 in block 2, 650 in block 5
            sinks = torch.from_numpy(sinks_np.astype(np.int32)).cuda()
            keep = torch.tensor([1, 0, 0, 0, 1, 1], dtype=torch.uint8, device="cuda")
            fb.focus_sparse_attn(ctx, sh, Qz, s.M, nrow, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP, bidx, 2, bcnt,
                                 sinks, keep, 3, O, lse)
            got = fstep.from_device(O)
            for h in range(H):
                ks = fo.key_set(s.M, s.L, B, blocks[h // 2], sinks_np)
                assert max_abs(got[0, h], V[h // 2, ks].mean(axis=0)) < 4e-3
                assert abs(lse[h, 0].item() - math.log(len(ks))) < 1e-4
            # nothing kept from the prompt
            bcnt0 = torch.zeros(2, dtype=torch.int32, device="cuda")
            fb.focus_sparse_attn(ctx, sh, Qz, s.M, nrow, None, None, 0, dK, dV, fb.HEADS_PER_KV_GROUP, bidx, 2, bcnt0,
                                 None, None, 0, O, lse)
            got = fstep.from_device(O)
            for h in range(H):
                assert max_abs(got[0, h], V[h // 2, s.M:].mean(axis=0)) < 4e-3
        ctx.set_force_simt(False)
    assert ctx.poll_status() == 0


def test_sink_blocks_mode_and_bad_indices_are_reported(ctx):
    w = small_workload("f32", 64, 64)
    s = w.shape
    host, dev = make_inputs(w)
    ora = oracle_chain(w, host, fb.HEADS_PER_KV_GROUP, fb.SINK_BLOCKS)
    b = fstep.StepBuffers(w, sink_mode=fb.SINK_BLOCKS)
    R = torch.from_numpy(ora["R"].astype(np.float32).reshape(-1)).cuda()
    b.sink_idx.copy_(torch.from_numpy(ora["sinks"].astype(np.int32)))
    fb.focus_select_blocks(ctx, b.shape, R, fb.HEADS_PER_KV_GROUP, w.C, b.sink_idx, w.n_sink, fb.SINK_BLOCKS,
                           b.block_idx, b.max_blocks, b.block_cnt, b.sink_keep)
    bi = b.block_idx.cpu().numpy().reshape(b.G, b.max_blocks)
    for g in range(b.G):
        n = b.block_cnt[g].item()
        assert bi[g, :n].tolist() == ora["blocks"][g].tolist() and (bi[g, n:] == -1).all()
    assert b.sink_keep.sum().item() == 0
    assert ctx.poll_status() == 0
    # a block index out of range is skipped and reported, not dereferenced
    b.block_idx[0] = 10 ** 6
    fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
    q_rows, n_rows, max_rows = b._rows()
    fb.focus_sparse_attn(ctx, b.shape, dev["Q"], s.M, s.N, q_rows, n_rows, max_rows, dev["K"], dev["V"],
                         fb.HEADS_PER_KV_GROUP, b.block_idx, b.max_blocks, b.block_cnt, b.sink_idx, b.sink_keep,
                         w.n_sink, b.O, b.lse)
    assert ctx.poll_status() == fb.ERR_INVALID_ARG
    assert ctx.poll_status() == 0


def test_host_side_argument_matrix(ctx):
    w = small_workload("f32", 64, 64)
    s = w.shape
    _, dev = make_inputs(w)
    b = fstep.StepBuffers(w)
    lib = ctx._lib
    import ctypes as C
    sh = b.shape
    st = torch.cuda.current_stream().cuda_stream
    p = lambda t: t.data_ptr()
    # k beyond the supported maximum, block range beyond the supported maximum
    assert lib.focus_select_queries(ctx.handle, p(dev["conf"]), p(dev["masked"]), s.L, 0, s.L, 5000, 8, 0, s.L,
                                    p(b.focus_idx), p(b.n_focus), p(b.active_idx), p(b.n_active), st) == fb.ERR_UNSUPPORTED
    assert lib.focus_select_queries(ctx.handle, p(dev["conf"]), p(dev["masked"]), s.L, 5, 3, 4, 8, 0, s.L,
                                    p(b.focus_idx), p(b.n_focus), p(b.active_idx), p(b.n_active), st) == fb.ERR_INVALID_ARG
    # C > nb
    assert lib.focus_select_blocks(ctx.handle, C.byref(sh), p(b.R), 0, s.nb + 1, p(b.sink_idx), w.n_sink, 0,
                                   p(b.block_idx), s.nb + 1, p(b.block_cnt), p(b.sink_keep), st) == fb.ERR_INVALID_ARG
    # both / neither of K and Kbar
    assert lib.focus_score_blocks(ctx.handle, C.byref(sh), p(dev["Q"]), s.M, p(b.focus_idx), p(b.n_focus), w.k,
                                  None, None, 0, p(b.R), st) == fb.ERR_INVALID_ARG
    # head_dim the kernels are not built for
    bad = fb.make_shape(s.L, s.M, 4, 4, 96, 64, fb.F32)
    assert lib.focus_dense_attn(ctx.handle, C.byref(bad), p(dev["Q"]), s.M, s.N, None, None, 0, p(dev["K"]),
                                p(dev["V"]), p(b.O), None, st) == fb.ERR_UNSUPPORTED
    # workspace too small is reported, not overrun
    tiny = fb.Context(0, workspace_bytes=4096)
    assert tiny._lib.focus_find_sinks(tiny.handle, C.byref(sh), p(dev["Q"]), s.M, p(b.active_idx), p(b.n_active),
                                      b.max_active, p(dev["K"]), None, w.n_sink, 0, s.M, p(b.sink_idx), None,
                                      st) == fb.ERR_WORKSPACE_TOO_SMALL
    tiny.close()


def test_misaligned_tensors_are_refused_on_the_host(ctx):
    """A tensor that does not start on a 16-byte boundary is turned away before anything is launched (the kernels use
    128-bit loads and TMA copies, which would fault on it)."""
    w = small_workload("bf16", 128, 128)
    s = w.shape
    host, dev = make_inputs(w)
    b = fstep.StepBuffers(w)
    fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
    off = lambda t: torch.cat([t.reshape(-1), t.reshape(-1)[:8]])[1:]          # same values, start + 2 bytes
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    n0 = fb.focus_launch_count()
    calls = [
        lambda: fb.focus_dense_attn(ctx, b.shape, off(dev["Q"]), s.M, s.N, None, None, 0, dev["K"], dev["V"], b.O, b.lse),
        lambda: fb.focus_dense_attn(ctx, b.shape, dev["Q"], s.M, s.N, None, None, 0, off(dev["K"]), dev["V"], b.O, b.lse),
        lambda: fb.focus_dense_attn(ctx, b.shape, dev["Q"], s.M, s.N, None, None, 0, dev["K"], off(dev["V"]), b.O, b.lse),
        lambda: fb.focus_dense_attn(ctx, b.shape, dev["Q"], s.M, s.N, None, None, 0, dev["K"], dev["V"], off(b.O), b.lse),
        lambda: fstep.find_sinks(ctx, b, dev["Q"], off(dev["K"]), None),
        lambda: fb.focus_pool_keys(ctx, b.shape, off(dev["K"]), Kbar),
        lambda: fb.focus_score_blocks(ctx, b.shape, off(dev["Q"]), s.M, b.focus_idx, b.n_focus, w.k, dev["K"], None, 0, b.R),
        lambda: fstep.sparse_layer(ctx, b, dev["Q"], dev["K"], off(dev["V"]), Kbar=Kbar),
        lambda: fb.focus_update_kv(ctx, b.shape, dev["K"].clone(), dev["V"].clone(),
                                   off(torch.zeros(b.max_active, s.Hkv, s.d, dtype=torch.bfloat16, device="cuda")),
                                   torch.zeros(b.max_active, s.Hkv, s.d, dtype=torch.bfloat16, device="cuda"),
                                   b.active_idx, b.n_active, b.max_active),
    ]
    for call in calls:
        with pytest.raises(fb.FocusError) as e:
            call()
        assert e.value.code == fb.ERR_INVALID_ARG
    assert fb.focus_launch_count() == n0
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("merge", [None, "counters", "kernel"])
@pytest.mark.parametrize("cfg", [SHAPES[1], SHAPES[3], SHAPES[5]])
def test_a_context_of_exactly_the_advertised_workspace_runs_every_stage(cfg, merge):
    """focus_workspace_bytes is a promise: a context created with that many bytes must carry every call on the
    shape — sink identification with and without a log-sum-exp from a dense pass, pooling, cold and warm scoring,
    selection, attention in both row modes, the fused layer — also when the key splits merge through global
    memory (forced)."""
    dtype, d, B, H, Hkv = cfg
    w = small_workload(dtype, d, B, H=H, Hkv=Hkv, L=5200, M=4500, n_sink=150, C=9, seed=12)
    s = w.shape
    host, dev = make_inputs(w)
    need = fb.focus_workspace_bytes(fstep.c_shape(s), s.N, w.C, w.n_sink)
    c = fb.Context(0, workspace_bytes=need)
    if merge:
        c.set_option(fb.OPT_MERGE_MODE, fb.MERGE_COUNTERS if merge == "counters" else fb.MERGE_KERNEL)
    try:
        Kbar = torch.zeros(Hkv, s.nb, d, dtype=torch.float32, device="cuda")
        for rows in ("active", "gen"):
            b = fstep.StepBuffers(w, rows=rows)
            fstep.select_queries(c, b, dev["conf"], dev["masked"])
            fstep.dense_layer(c, b, dev["Q"], dev["K"], dev["V"])
            fstep.find_sinks(c, b, dev["Q"], dev["K"], None)
            no_lse = b.sink_idx.clone()
            if rows == "active":
                fstep.find_sinks(c, b, dev["Q"], dev["K"], b.lse)
                assert torch.equal(no_lse, b.sink_idx)
            fb.focus_pool_keys(c, b.shape, dev["K"], Kbar)
            fstep.sparse_layer(c, b, dev["Q"], dev["K"], dev["V"], Kbar=None, fused=False)       # cold scoring
            cold = b.O.clone()
            fstep.sparse_layer(c, b, dev["Q"], dev["K"], dev["V"], Kbar=Kbar, fused=False)
            fstep.sparse_layer(c, b, dev["Q"], dev["K"], dev["V"], Kbar=Kbar, fused=True)
            torch.cuda.synchronize()
            assert c.poll_status() == 0
            assert (cold.float() - b.O.float()).abs().max().item() <= 2e-2
    finally:
        c.close()


@pytest.mark.parametrize("case", ["all_equal", "duplicated_keys", "random"])
def test_sink_selection_on_a_long_candidate_range(ctx, case):
    """A candidate range long enough for the multi-CTA selection (16 000 prompt positions).  The selected set must be
    exactly the n_sink largest of the scores the library itself reports, equal scores taken in index order
    ("all_equal": Q = 0, every score is 1/L, the set is the first n_sink positions; "duplicated_keys": every score
    value occurs four times or more, so the threshold cuts a run of equal scores), and agree with the oracle outside
    the near-threshold band."""
    L, M, H, d, n_sink, n_act = 16384, 16000, 2, 128, 161, 24
    s = wl.Shape(L, M, H, H, d, 128, "bf16")
    rng = np.random.default_rng(11)
    K = rng.standard_normal((H, L, d)).astype(np.float32) / math.sqrt(d)
    if case == "duplicated_keys":
        K = K[:, np.arange(L) % 4000]
    Qf = rng.standard_normal((s.N, H, d)).astype(np.float32) / math.sqrt(d)
    if case == "all_equal":
        Qf[:] = 0.0
    Qs, Ks = wl.to_storage(Qf, "bf16"), wl.to_storage(np.ascontiguousarray(K), "bf16")
    dQ, dK = fstep.to_device(Qs, "bf16"), fstep.to_device(Ks, "bf16")
    active = np.sort(rng.choice(np.arange(M, L), size=n_act, replace=False)).astype(np.int32)
    d_active = torch.from_numpy(active).cuda()
    d_nact = torch.tensor([n_act], dtype=torch.int32, device="cuda")
    sink_idx = torch.full((n_sink,), -7, dtype=torch.int32, device="cuda")
    scores = torch.zeros(L, dtype=torch.float32, device="cuda")
    fb.focus_find_sinks(ctx, fstep.c_shape(s), dQ, M, d_active, d_nact, n_act, dK, None, n_sink, 0, M, sink_idx, scores)
    assert ctx.poll_status() == 0
    got = sink_idx.cpu().numpy()
    sc = scores.cpu().numpy()
    # exact selection on the library's own float32 scores, ties to the lower index
    order = np.argsort(-sc[:M].astype(np.float64), kind="stable")[:n_sink]
    assert np.array_equal(got, np.sort(order))
    if case == "all_equal":
        assert np.array_equal(got, np.arange(n_sink))
    if case == "duplicated_keys":
        tau = sc[got].min()
        assert (sc[:M] == tau).sum() > (sc[got] == tau).sum() >= 1, "the threshold was meant to cut a run of equal scores"
    # oracle parity outside the band
    Q64, K64 = wl.storage_to_f64(Qs, "bf16"), wl.storage_to_f64(Ks, "bf16")
    S = fo.sink_scores(Q64[active - M], K64, 1.0 / math.sqrt(d))
    ref = fo.find_sinks(S, n_sink, 0, M)
    assert np.max(np.abs(sc - S)) <= 2e-3 * np.max(S)
    check_topk_band(got, ref, S, range(M), 1e-3, what="sink_idx")


@pytest.mark.parametrize("nb,C", [(700, 37), (257, 256), (3000, 1), (1022, 31)])
def test_block_selection_with_many_blocks_and_cut_ties(ctx, nb, C):
    """Top-C over several hundred to a few thousand blocks (the radix path of the selection kernels), scores
    quantised so that the threshold cuts a run of equal scores: the set must be the oracle's exactly (float32 scores
    are given, nothing is recomputed), equal scores taken in block order, and the keep flags must follow it.  Runs the
    stand-alone stage and, where the pooled keys reproduce the scores, the fused layer's selection."""
    B, G = 64, 3
    M = nb * B - 17                                      # short last block
    s = wl.Shape(M + 192, M, G, G, 64, B, "f32")
    assert s.nb == nb
    rng = np.random.default_rng(nb + C)
    R = rng.integers(0, 23, size=(G, nb)).astype(np.float32) / 7.0 - 1.0     # 23 distinct values, signs mixed
    R[1, ::5] = -0.0
    sinks = np.sort(rng.choice(M, size=40, replace=False)).astype(np.int32)
    blocks, keep = fo.select_blocks(R, C, sinks, B)
    dR = torch.from_numpy(R.reshape(-1)).cuda()
    d_sinks = torch.from_numpy(sinks).cuda()
    bidx = torch.full((G * C,), -9, dtype=torch.int32, device="cuda")
    bcnt = torch.zeros(G, dtype=torch.int32, device="cuda")
    skeep = torch.full((G * 40,), 7, dtype=torch.uint8, device="cuda")
    fb.focus_select_blocks(ctx, fstep.c_shape(s), dR, fb.HEADS_PER_KV_GROUP, C, d_sinks, 40, fb.SINK_TOKENS, bidx, C, bcnt,
                           skeep)
    assert ctx.poll_status() == 0
    got = bidx.cpu().numpy().reshape(G, C)
    for g in range(G):
        assert bcnt[g].item() == C
        assert got[g].tolist() == blocks[g].tolist(), f"group {g}"
        tau = R[g, blocks[g]].min()
        if C < nb:
            assert (R[g] == tau).sum() > (R[g, blocks[g]] == tau).sum() >= 1, "the threshold was meant to cut a tie"
    assert np.array_equal(skeep.cpu().numpy().reshape(G, 40), keep)


@pytest.mark.parametrize("case", ["small_active", "llada_8k_gen", "sweep_32k_gen", "block64_gen"])
def test_results_are_deterministic(ctx, case):
    """Same inputs, same bits, run after run: the small GQA shape on the one-warpgroup kernel, and full-size
    gen-row launches on the two-tile and key-pair forms with their in-cluster split merges."""
    if case == "small_active":
        w, rows = small_workload("bf16", 128, 128, H=8, Hkv=2), "active"
    elif case == "llada_8k_gen":
        w, rows = wl.config(1), "gen"
    elif case == "sweep_32k_gen":
        w, rows = wl.config(4, L=32768, keep_den=16), "gen"
    else:
        w, rows = small_workload("bf16", 128, 64, H=4, Hkv=4, L=9000, M=8744, n_sink=87, C=40), "gen"
    host, dev = make_inputs(w)
    outs = []
    for _ in range(3):
        b = fstep.StepBuffers(w, rows=rows)
        fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
        fstep.dense_layer(ctx, b, dev["Q"], dev["K"], dev["V"])
        dense = b.O.view(torch.int16).clone()
        fstep.find_sinks(ctx, b, dev["Q"], dev["K"], b.lse if rows == "active" else None)
        fstep.sparse_layer(ctx, b, dev["Q"], dev["K"], dev["V"])
        torch.cuda.synchronize()
        outs.append([t.clone() for t in (dense, b.sink_idx, b.sink_scores, b.R, b.block_idx, b.O.view(torch.int16), b.lse)])
    for other in outs[1:]:
        for a, c in zip(outs[0], other):
            assert torch.equal(a, c)
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("rows", ["active", "gen"])
def test_step_replayed_from_a_cuda_graph_matches_eager_calls(ctx, rows):
    """The benchmark times a step as one CUDA-graph replay (counts stay on the device, the kernels are chained by
    programmatic dependent launch).  A small step -- two dense layers, sink identification, three sparse layers with
    cached pooled keys -- captured into a graph must reproduce the eager calls bit for bit, replay after replay."""
    w = small_workload("bf16", 128, 128, H=8, Hkv=2, L=2600, M=2100, n_sink=21, C=5)
    host, dev = make_inputs(w)
    s = w.shape
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    b0 = fstep.StepBuffers(w, rows=rows)
    fb.focus_pool_keys(ctx, b0.shape, dev["K"], Kbar)
    n_layers = 5

    def step(b, outs):
        fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
        for l in range(2):
            fstep.dense_layer(ctx, b, dev["Q"], dev["K"], dev["V"], O=outs[l])
        if rows == "active":
            fstep.find_sinks(ctx, b, dev["Q"], dev["K"], b.lse)
        else:
            fstep.find_sinks(ctx, b, dev["Q"], dev["K"], None)
        for l in range(2, n_layers):
            fstep.sparse_layer(ctx, b, dev["Q"], dev["K"], dev["V"], Kbar=Kbar, O=outs[l])

    def fresh():
        b = fstep.StepBuffers(w, rows=rows)
        outs = [torch.zeros_like(b.O) for _ in range(n_layers)]
        return b, outs

    b_e, o_e = fresh()
    step(b_e, o_e)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    b_g, o_g = fresh()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(b_g, o_g)                                   # warm-up outside the capture (attributes, lazy set-up)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(b_g, o_g)
    for _ in range(3):
        for t in o_g:
            t.zero_()
        b_g.sink_idx.fill_(-5); b_g.block_idx.fill_(-5)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        for a, c in zip(o_e, o_g):
            assert torch.equal(a.view(torch.int16), c.view(torch.int16))
        for name in ("sink_idx", "sink_scores", "block_idx", "block_cnt", "R", "lse", "active_idx", "focus_idx"):
            assert torch.equal(getattr(b_e, name), getattr(b_g, name)), name


@pytest.mark.parametrize("rows", ["active", "gen"])
def test_launch_options_change_nothing_but_the_launches(rows):
    """focus_set_option: without programmatic dependent launches (plain stream order: what a caller sets when a foreign
    kernel produces an input immediately before a fused layer) the same kernels run the same arithmetic, so a small
    step must come out bit for bit as by default; without the three-warpgroup kernels the one-tile kernel takes
    their launches and the outputs agree to rounding, index sets exactly."""
    w = small_workload("bf16", 128, 128, H=8, Hkv=2, L=2600, M=2100, n_sink=21, C=5)
    host, dev = make_inputs(w)
    s = w.shape
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    runs = {}
    for name, opts in (("default", []), ("no_pdl", [(fb.OPT_NO_PDL, 1)]), ("no_wide", [(fb.OPT_NO_WIDE, 1)])):
        c = fb.Context(0)
        try:
            for o, v in opts:
                assert c.set_option(o, v) == 0
            b = fstep.StepBuffers(w, rows=rows)
            fb.focus_pool_keys(c, b.shape, dev["K"], Kbar)
            fstep.select_queries(c, b, dev["conf"], dev["masked"])
            outs = []
            for l in range(2):
                fstep.dense_layer(c, b, dev["Q"], dev["K"], dev["V"])
                outs.append(b.O.clone())
            variants = [c.last_attn_variant()]
            fstep.find_sinks(c, b, dev["Q"], dev["K"], b.lse if rows == "active" else None)
            for l in range(3):
                fstep.sparse_layer(c, b, dev["Q"], dev["K"], dev["V"], Kbar=Kbar)
                outs.append(b.O.clone())
            variants.append(c.last_attn_variant())
            torch.cuda.synchronize()
            assert c.poll_status() == 0
            runs[name] = dict(outs=outs, sinks=b.sink_idx.clone(), blocks=b.block_idx.clone(), keep=b.sink_keep.clone(),
                              lse=b.lse.clone(), variants=variants)
        finally:
            c.close()
    d, p, nw = runs["default"], runs["no_pdl"], runs["no_wide"]
    assert p["variants"] == d["variants"]
    for a, z in zip(d["outs"], p["outs"]):
        assert torch.equal(a.view(torch.int16), z.view(torch.int16))
    assert torch.equal(d["lse"], p["lse"])
    for r in (p, nw):
        assert torch.equal(d["sinks"], r["sinks"]) and torch.equal(d["blocks"], r["blocks"]) and torch.equal(d["keep"], r["keep"])
    assert nw["variants"] == [2, 2]
    if rows == "gen":
        assert d["variants"][0] in (3, 4), "the default dense layer was meant to take a three-warpgroup kernel"
    for a, z in zip(d["outs"], nw["outs"]):
        assert max_abs(fstep.from_device(a), fstep.from_device(z)) <= 2e-2


def test_step_with_nothing_left_to_unmask(ctx):
    """No masked position in the decoding block: I_focus and I_active are empty.  The attention calls have no rows to
    compute (outputs stay untouched), sink identification and the fused layer report the undefined inputs through
    the status word instead of reading or writing out of range, and the context stays usable."""
    w = small_workload("bf16", 128, 128, H=4, Hkv=4)
    host, dev = make_inputs(w)
    b = fstep.StepBuffers(w)
    masked = torch.zeros_like(dev["masked"])
    fstep.select_queries(ctx, b, dev["conf"], masked)
    assert b.n_focus.item() == 0 and b.n_active.item() == 0
    assert (b.focus_idx == -1).all() and (b.active_idx == -1).all()
    b.O.fill_(3.0); b.lse.fill_(-7.0)
    fstep.dense_layer(ctx, b, dev["Q"], dev["K"], dev["V"])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    assert (b.O == 3.0).all() and (b.lse == -7.0).all()
    fstep.find_sinks(ctx, b, dev["Q"], dev["K"], b.lse)
    assert ctx.poll_status() == fb.ERR_INVALID_ARG          # scores are undefined without active rows
    assert (b.sink_idx == -1).all()
    Kbar = torch.zeros(w.shape.Hkv, w.shape.nb, w.shape.d, dtype=torch.float32, device="cuda")
    fb.focus_pool_keys(ctx, b.shape, dev["K"], Kbar)
    fstep.sparse_layer(ctx, b, dev["Q"], dev["K"], dev["V"], Kbar=Kbar)
    torch.cuda.synchronize()
    assert ctx.poll_status() == fb.ERR_INVALID_ARG          # no focus query to score blocks with
    assert (b.O == 3.0).all()
    # the same context still computes a normal step afterwards
    fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
    fstep.dense_layer(ctx, b, dev["Q"], dev["K"], dev["V"])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0 and b.n_active.item() > 0


@pytest.mark.parametrize("merge", ["counters", "kernel"])
def test_split_merge_fallbacks_match_the_default(merge, ctx):
    """When the clusters of a launch would not all be resident, the key splits of a query tile are merged through
    global memory: by the CTA that arrives last at the tile's counter, or by a separate kernel.  Both fallbacks are
    forced here (focus_set_option on a second context) and must agree with the oracle and, to the last bf16 digit
    or the one next to it, with the default path."""
    w = small_workload("bf16", 128, 128, H=4, Hkv=2, L=5200, M=4500, n_sink=45, C=9)
    host, dev = make_inputs(w)
    other = fb.Context(0)
    assert other.set_option(fb.OPT_MERGE_MODE, fb.MERGE_COUNTERS if merge == "counters" else fb.MERGE_KERNEL) == 0
    try:
        outs = []
        for c in (ctx, other):
            b = fstep.StepBuffers(w)
            fstep.select_queries(c, b, dev["conf"], dev["masked"])
            n0 = fb.focus_launch_count()
            fstep.dense_layer(c, b, dev["Q"], dev["K"], dev["V"])
            n_launch = fb.focus_launch_count() - n0
            # one kernel when the merge runs inside the attention kernel, two with the separate combine kernel
            assert n_launch == (2 if (c is other and merge == "kernel") else 1)
            dense_O, dense_lse = b.O.clone(), b.lse.clone()
            fstep.find_sinks(c, b, dev["Q"], dev["K"], b.lse)
            fstep.sparse_layer(c, b, dev["Q"], dev["K"], dev["V"])
            torch.cuda.synchronize()
            assert c.poll_status() == 0
            outs.append((dense_O, dense_lse, b.O.clone(), b.lse.clone(), b.sink_idx.clone(), b.block_idx.clone(), b))
        a, o = outs
        assert torch.equal(a[4], o[4]) and torch.equal(a[5], o[5])
        for i in (0, 2):
            assert (a[i].float() - o[i].float()).abs().max().item() <= 2 ** -8 * a[i].float().abs().max().item()
        for i in (1, 3):
            assert (a[i] - o[i]).abs().max().item() <= 1e-5
        # and against the oracle (dense layer, all heads)
        b = o[6]
        na = b.n_active.item()
        act = b.active_idx.cpu().numpy()[:na]
        Q, K, V = host["Q"], host["K"], host["V"]
        Od, ld = fo.dense_attn(Q[act - w.shape.M], K, V, 1.0 / math.sqrt(w.shape.d))
        got = fstep.from_device(o[0])[:na]
        assert max_abs(got, Od) <= TOL_ABS["bf16"] and rel_rms(got, Od) <= TOL_RMS["bf16"]
    finally:
        other.close()


def test_a_wait_that_nothing_satisfies_gives_up_and_is_reported(ctx):
    """Every barrier wait in the tensor-core kernels is bounded.  The library's self-test lets one CTA wait two
    milliseconds on a barrier nobody arrives at: it must come back (well inside a second), the status word must say
    TIMEOUT, and the context must go on working."""
    import time
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ctx.selftest_bounded_wait(2000)
    status = ctx.poll_status()                          # synchronises the stream
    dt = time.perf_counter() - t0
    assert status == fb.ERR_TIMEOUT
    assert dt < 1.0
    assert ctx.poll_status() == 0                       # polled once, cleared
    w = small_workload("bf16", 128, 128)
    host, dev = make_inputs(w)
    b = fstep.StepBuffers(w)
    fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
    fstep.dense_layer(ctx, b, dev["Q"], dev["K"], dev["V"])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0 and b.n_active.item() > 0


@pytest.mark.parametrize("cfg", [SHAPES[0], SHAPES[3]])
def test_compact_query_rows_give_the_same_step(ctx, cfg):
    """A caller that holds only the I_active rows of Q (gathered in list order) and hands the library local row numbers
    gets, bit for bit, what a caller with every gen row of Q and absolute positions gets: dense layer, sink set,
    sparse layer."""
    dtype, d, B, H, Hkv = cfg
    w = small_workload(dtype, d, B, H=H, Hkv=Hkv, L=2300, M=1900, n_sink=30, C=5, seed=19)
    s = w.shape
    host, dev = make_inputs(w)
    outs = []
    for rows in ("active", "compact"):
        b = fstep.StepBuffers(w, rows=rows)
        fstep.select_queries(ctx, b, dev["conf"], dev["masked"])
        Q = dev["Q"]
        if rows == "compact":
            na, nf = b.n_active.item(), b.n_focus.item()
            act, foc = b.active_idx.cpu().numpy()[:na], b.focus_idx.cpu().numpy()[:nf]
            b.set_local_focus(foc, act)
            Q = torch.zeros(b.max_active, H, d, dtype=dev["Q"].dtype, device="cuda")
            Q[:na] = dev["Q"][torch.from_numpy(act - s.M).cuda().long()]
        Kbar = torch.zeros(Hkv, s.nb, d, dtype=torch.float32, device="cuda")
        fb.focus_pool_keys(ctx, b.shape, dev["K"], Kbar)
        fstep.dense_layer(ctx, b, Q, dev["K"], dev["V"])
        dense_O, dense_lse = b.O.clone(), b.lse.clone()
        fstep.find_sinks(ctx, b, Q, dev["K"], b.lse)
        fstep.sparse_layer(ctx, b, Q, dev["K"], dev["V"], Kbar=Kbar)
        torch.cuda.synchronize()
        outs.append((dense_O, dense_lse, b.sink_idx.clone(), b.block_idx.clone(), b.sink_keep.clone(), b.O.clone(),
                     b.lse.clone()))
    for x, y in zip(*outs):
        assert torch.equal(x, y)
    assert ctx.poll_status() == 0
