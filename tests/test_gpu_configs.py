"""GPU parity on the five benchmark configurations at their full sizes, through the C ABI, in the launch
configuration the benchmark uses.  Index sets are compared in full: the query sets exactly, the sink set of every
step and the block set of EVERY KV group of EVERY sparse layer / step / sweep point against the oracle's scores
with the near-threshold band rule.  Attention outputs are compared on sampled (layer, head) pairs that the oracle
computes one by one, with the oracle given the index sets the GPU chose (after those have been validated), so that
a legitimate in-band difference of a set does not masquerade as an attention error.

How many candidates sat inside the band of each check is collected in BAND_LOG and, when the environment variable
FOCUS_BAND_REPORT names a file, written there as JSON at the end of the module (the band-occupancy table of the
results document comes from it)."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import focus_oracle as fo
from paper_2602_02159_b200 import binding as fb
from paper_2602_02159_b200 import step as fstep
from paper_2602_02159_b200 import workloads as wl
from tests.helpers import check_topk_band, max_abs, rel_rms

pytestmark = pytest.mark.gpu

TOL_ABS = {"f32": 1e-5, "bf16": 2e-2}
TOL_RMS = {"f32": 1e-5, "bf16": 1e-2}
BAND = 1e-3


BAND_LOG = []      # (case, stage, layer/step, group, candidates in band, set size, candidates)


def log_band(case, stage, where, group, band, k, n_cand):
    BAND_LOG.append({"case": case, "stage": stage, "where": where, "group": group, "in_band": int(band),
                     "set_size": int(k), "candidates": int(n_cand)})


@pytest.fixture(scope="module")
def ctx():
    c = fb.Context(0, workspace_bytes=512 << 20)
    yield c
    assert c.poll_status() == 0
    c.close()
    path = os.environ.get("FOCUS_BAND_REPORT")
    if path:
        with open(path, "w") as f:
            json.dump(BAND_LOG, f)


def f64(a, dtype, sl=slice(None)):
    return wl.storage_to_f64(a[sl], dtype)


def oracle_sinks_by_head(Qa_store, K_store, dtype, scale):
    """S_j (Eq. 6) accumulated head by head to bound host memory (S is a mean over heads)."""
    H, Hkv = Qa_store.shape[1], K_store.shape[0]
    hpg = H // Hkv
    acc = None
    for g in range(Hkv):
        Sg = fo.sink_scores(f64(Qa_store[:, g * hpg:(g + 1) * hpg], dtype), f64(K_store, dtype, slice(g, g + 1)), scale)
        acc = Sg if acc is None else acc + Sg
    return acc / Hkv


def check_sinks_exact_on_own_scores(sink_idx_gpu, S_gpu, n_sink, M, what):
    """Complement of the band rule: on the float32 scores the GPU itself produced, its Top-n with the tie rule must be
    exact -- whatever the band forgives, it forgives score rounding, never the selection."""
    own = fo.find_sinks(np.asarray(S_gpu, dtype=np.float64), n_sink, 0, M)
    assert [int(i) for i in sink_idx_gpu if i >= 0] == own.tolist(), f"{what}: selection differs on the GPU's own scores"


def check_block_sets(w, t, b_blocks, b_keep, sinks, focus, case, where):
    """Block set and sink-keep flags of EVERY KV group of one sparse layer against the oracle (Eq. 7, Top-C, Eq. 8):
    the oracle scores one group at a time (one mean-pool of that group's prompt keys)."""
    s = w.shape
    hpg = s.H // s.Hkv
    for g in range(s.Hkv):
        K = f64(t["K"], s.dtype, slice(g, g + 1))
        Qf = f64(t["Q"][focus - s.M][:, g * hpg:(g + 1) * hpg], s.dtype)
        R = fo.score_blocks(Qf, fo.pool_keys(K, s.M, s.B), fo.PER_KV_GROUP)
        ora_blocks, _ = fo.select_blocks(R, w.C, sinks, s.B)
        band = check_topk_band(b_blocks[g], ora_blocks[0], R[0], range(s.nb), BAND, scale_ref=np.abs(R[0]).max(),
                               what=f"{case} {where}: blocks of group {g}")
        log_band(case, "blocks", where, g, band, w.C, s.nb)
        mine = {int(x) for x in b_blocks[g] if x >= 0}
        assert b_keep[g].tolist() == [0 if (int(j) // s.B) in mine else 1 for j in sinks], f"{case} {where}: keep flags {g}"


def check_layer(w, t, b_blocks, b_keep, sinks, focus, active, O_gpu, lse_gpu, heads, rows_pos, dense=False):
    """Attention outputs of sampled heads of one layer; the oracle attends over the key set the GPU chose (its block
    sets are validated for every group by check_block_sets)."""
    s = w.shape
    hpg = s.H // s.Hkv
    scale = 1.0 / math.sqrt(s.d)
    for h in heads:
        g = h // hpg
        K = f64(t["K"], s.dtype, slice(g, g + 1))
        V = f64(t["V"], s.dtype, slice(g, g + 1))
        Q = f64(t["Q"][:, g * hpg:(g + 1) * hpg], s.dtype)
        if dense:
            O, lse = fo.dense_attn(Q[rows_pos - s.M][:, [h - g * hpg]], K, V, scale)
        else:
            blocks_g = np.array([x for x in b_blocks[g] if x >= 0])
            O, lse = fo.sparse_attn(Q[rows_pos - s.M][:, [h - g * hpg]], K, V, s.M, s.B, [blocks_g], sinks, scale)
        got = O_gpu[:len(rows_pos), h]
        assert max_abs(got, O[:, 0]) <= TOL_ABS[s.dtype], f"head {h}"
        assert rel_rms(got, O[:, 0]) <= TOL_RMS[s.dtype], f"head {h}"
        assert max_abs(lse_gpu[h, :len(rows_pos)], lse[0]) <= 2e-3


def run_selection(ctx, w, b, conf, masked):
    fstep.select_queries(ctx, b, torch.from_numpy(conf).cuda(), torch.from_numpy(masked).cuda())
    s = w.shape
    focus, active = fo.select_queries(conf, masked, w.blk_lo, w.blk_hi, w.k, w.w, s.M, s.L)
    assert b.n_focus.item() == len(focus) and b.n_active.item() == len(active)
    assert b.focus_idx.cpu().numpy()[:len(focus)].tolist() == focus.tolist()
    assert b.active_idx.cpu().numpy()[:len(active)].tolist() == active.tolist()
    return focus, active


def single_layer_case(ctx, w, rows, heads, head_reduce=fb.HEADS_PER_KV_GROUP, sink_mode=fb.SINK_TOKENS,
                      check_dense=True, variant="fix"):
    """Whole chain of one layer: select_queries -> dense (+LSE) -> find_sinks -> sparse layer."""
    s = w.shape
    t = wl.gen_qkv(s, w.seed, variant=variant)
    c_prev, _ = wl.gen_confidence(w.seed, s.N)
    conf, masked = wl.full_conf(s, c_prev), wl.gen_masked(w)
    dQ, dK, dV = (fstep.to_device(t[n], s.dtype) for n in "QKV")
    scale = 1.0 / math.sqrt(s.d)
    ba = fstep.StepBuffers(w, rows="active", head_reduce=head_reduce, sink_mode=sink_mode)
    focus, active = run_selection(ctx, w, ba, conf, masked)
    fstep.dense_layer(ctx, ba, dQ, dK, dV)
    if check_dense and head_reduce == fb.HEADS_PER_KV_GROUP:
        check_layer(w, t, None, None, None, focus, active, fstep.from_device(ba.O), fstep.from_device(ba.lse), heads,
                    active, dense=True)
    fstep.find_sinks(ctx, ba, dQ, dK, ba.lse)
    S = oracle_sinks_by_head(t["Q"][active - s.M], t["K"], s.dtype, scale)
    sinks = fo.find_sinks(S, w.n_sink, 0, s.M)
    band = check_topk_band(ba.sink_idx.cpu().numpy(), sinks, S, range(s.M), BAND, what="sinks")
    case = f"{w.name}/{rows}" + ("" if variant == "fix" else f"/{variant}")
    log_band(case, "sinks", "layer 0", -1, band, w.n_sink, s.M)
    S_gpu = fstep.from_device(ba.sink_scores)
    assert np.max(np.abs(S_gpu - S) / S) < 2e-3
    check_sinks_exact_on_own_scores(ba.sink_idx.cpu().numpy(), S_gpu, w.n_sink, s.M, case)
    planted = set(t["sink_pos"].tolist())
    sinks_gpu = ba.sink_idx.cpu().numpy()
    if variant == "fix":
        assert planted <= set(sinks_gpu.tolist()), "planted sinks not recovered"
    b = ba if rows == "active" else fstep.StepBuffers(w, rows="gen", head_reduce=head_reduce, sink_mode=sink_mode)
    if b is not ba:
        run_selection(ctx, w, b, conf, masked)
        b.sink_idx.copy_(ba.sink_idx)
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    fb.focus_pool_keys(ctx, b.shape, dK, Kbar)
    fstep.sparse_layer(ctx, b, dQ, dK, dV, Kbar=Kbar)
    torch.cuda.synchronize()
    rows_pos = active if rows == "active" else np.arange(s.M, s.L)
    G = b.G
    bi = b.block_idx.cpu().numpy().reshape(G, b.max_blocks)
    keep = b.sink_keep.cpu().numpy().reshape(G, -1)[:, :w.n_sink]
    if head_reduce == fb.HEADS_PER_KV_GROUP and sink_mode == fb.SINK_TOKENS:
        check_block_sets(w, t, bi, keep, sinks_gpu, focus, case, "layer 0")
        check_layer(w, t, bi, keep, sinks_gpu, focus, active, fstep.from_device(b.O), fstep.from_device(b.lse), heads,
                    rows_pos)
    else:
        # variants: one shared list (Eq. 7 as printed) and/or sink blocks; full oracle, small shapes only
        Q, K, V = (f64(t[n], s.dtype) for n in "QKV")
        R = fo.score_blocks(Q[focus - s.M], fo.pool_keys(K, s.M, s.B), head_reduce)
        ob, okeep = fo.select_blocks(R, w.C, sinks_gpu, s.B, sink_mode)
        for g in range(G):
            n = b.block_cnt[g].item()
            if sink_mode == fb.SINK_TOKENS:
                check_topk_band(bi[g], ob[g], R[g], range(s.nb), BAND, scale_ref=np.abs(R[g]).max())
            else:
                assert bi[g, :n].tolist() == ob[g].tolist()
        blocks = [np.array([x for x in bi[g] if x >= 0]) for g in range(G)]
        O, lse = fo.sparse_attn(Q[rows_pos - s.M], K, V, s.M, s.B, blocks, sinks_gpu, scale, heads=heads)
        got = fstep.from_device(b.O)[:len(rows_pos)]
        assert max_abs(got[:, heads], O[:, heads]) <= TOL_ABS[s.dtype]
        assert rel_rms(got[:, heads], O[:, heads]) <= TOL_RMS[s.dtype]
    assert ctx.poll_status() == 0
    return band


# ---- config 0: tiny fp32 step, every head, both query-row readings and the mode variants ---------------
@pytest.mark.parametrize("rows", ["active", "gen"])
def test_config0_tiny_f32(ctx, rows):
    w = wl.config(0)
    single_layer_case(ctx, w, rows, heads=list(range(w.shape.H)))


def test_config0_variants_all_heads_and_sink_blocks(ctx):
    import dataclasses
    w = wl.config(0)
    single_layer_case(ctx, w, "active", heads=list(range(8)), head_reduce=fb.HEADS_ALL)
    w2 = dataclasses.replace(w, n_sink=2)
    single_layer_case(ctx, w2, "active", heads=list(range(8)), sink_mode=fb.SINK_BLOCKS)


# ---- config 1: LLaDA-8B shape, one layer, one step --------------------------------------------------------
@pytest.mark.parametrize("rows", ["active", "gen"])
def test_config1_llada_8k(ctx, rows):
    w = wl.config(1)
    single_layer_case(ctx, w, rows, heads=[0, 9, 31])


# ---- config 2: full 32-layer step at 32K --------------------------------------------------------------------
def test_config2_full_32_layer_step(ctx):
    w = wl.config(2)
    s = w.shape
    NL, probe = w.n_layers, w.probe_layer
    check_layers = {0: [3], probe: [0, 31], probe + 1: [0, 17], NL - 1: [30]}
    c_prev, _ = wl.gen_confidence(w.seed, s.N)
    conf, masked = wl.full_conf(s, c_prev), wl.gen_masked(w)
    b = fstep.StepBuffers(w, rows="active")
    focus, active = run_selection(ctx, w, b, conf, masked)
    na = len(active)
    kept = {}
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    scale = 1.0 / math.sqrt(s.d)
    sinks_gpu = None
    for l in range(NL):
        t = wl.gen_qkv(s, l)                       # per-layer Q/K/V seeded by the layer index
        dQ, dK, dV = (fstep.to_device(t[n], s.dtype) for n in "QKV")
        if l <= probe:
            fstep.dense_layer(ctx, b, dQ, dK, dV)
            if l == probe:
                fstep.find_sinks(ctx, b, dQ, dK, b.lse)
                S = oracle_sinks_by_head(t["Q"][active - s.M], t["K"], s.dtype, scale)
                sinks = fo.find_sinks(S, w.n_sink, 0, s.M)
                band = check_topk_band(b.sink_idx.cpu().numpy(), sinks, S, range(s.M), BAND, what="sinks")
                log_band(w.name, "sinks", f"layer {l}", -1, band, w.n_sink, s.M)
                sinks_gpu = b.sink_idx.cpu().numpy()
                check_sinks_exact_on_own_scores(sinks_gpu, fstep.from_device(b.sink_scores), w.n_sink, s.M, w.name)
                assert set(t["sink_pos"].tolist()) <= set(sinks_gpu.tolist())
        else:
            fb.focus_pool_keys(ctx, b.shape, dK, Kbar)
            fstep.sparse_layer(ctx, b, dQ, dK, dV, Kbar=Kbar)
            torch.cuda.synchronize()
            bi = b.block_idx.cpu().numpy().reshape(b.G, b.max_blocks)
            keep = b.sink_keep.cpu().numpy().reshape(b.G, -1)[:, :w.n_sink]
            check_block_sets(w, t, bi, keep, sinks_gpu, focus, w.name, f"layer {l}")     # all 32 groups of every sparse layer
        if l in check_layers:
            torch.cuda.synchronize()
            bi = b.block_idx.cpu().numpy().reshape(b.G, b.max_blocks)
            keep = b.sink_keep.cpu().numpy().reshape(b.G, -1)[:, :w.n_sink]
            check_layer(w, t, bi, keep, sinks_gpu, focus, active, fstep.from_device(b.O), fstep.from_device(b.lse),
                        check_layers[l], active, dense=l <= probe)
        del t, dQ, dK, dV
    assert na > 0 and ctx.poll_status() == 0


def test_config2_one_layer_with_all_gen_rows(ctx):
    """The gen-row figures of the benchmark (512 query rows, 32 heads, 32K keys): one layer of config 2 with the whole
    gen region as query set -- dense on the two-tile form, sparse on the key-pair form."""
    single_layer_case(ctx, wl.config(2), "gen", heads=[0, 19])


def test_config3_one_layer_with_all_gen_rows(ctx):
    """Config 3 with the whole gen region as query set: 256 rows x 7 query heads per KV head stacked on each K/V tile."""
    single_layer_case(ctx, wl.config(3), "gen", heads=[0, 13, 27])


# ---- config 3: Dream-like GQA, 16 consecutive steps with AR(1) confidences ------------------------------------
def test_config3_gqa_16_steps(ctx):
    """Sixteen consecutive steps with the decoding state (confidence vector, masked set, token ids) resident on the
    device: every step ends with focus_commit_step, nothing of the state crosses to the host between steps.  The
    oracle drives its own copy of the state from the same synthetic confidence process; focus / active sets, sink
    and block sets, the unmasked positions and the final state are compared step by step."""
    w = wl.config(3)
    s = w.shape
    t = wl.gen_qkv(s, w.seed)
    dQ, dK, dV = (fstep.to_device(t[n], s.dtype) for n in "QKV")
    scale = 1.0 / math.sqrt(s.d)
    b = fstep.StepBuffers(w, rows="active")
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    fb.focus_pool_keys(ctx, b.shape, dK, Kbar)           # K/V are fixed over the steps: pooled once
    c_prev, c_cur = wl.gen_confidence(w.seed, s.N)
    # device-resident state and the oracle's own copy of it
    o_conf, o_masked, o_x = wl.full_conf(s, c_prev), wl.gen_masked(w), np.zeros(s.L, dtype=np.int32)
    d_conf, d_masked, d_x = (torch.from_numpy(a.copy()).cuda() for a in (o_conf, o_masked, o_x))
    picked, n_picked = torch.zeros(2, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda")
    gen_pos = list(range(s.M, s.L))
    hits = total = 0
    for step in range(w.n_steps):
        fstep.select_queries(ctx, b, d_conf, d_masked)
        focus, active = fo.select_queries(o_conf, o_masked, w.blk_lo, w.blk_hi, w.k, w.w, s.M, s.L)
        assert b.focus_idx.cpu().numpy()[:b.n_focus.item()].tolist() == focus.tolist()
        assert b.active_idx.cpu().numpy()[:b.n_active.item()].tolist() == active.tolist()
        fstep.dense_layer(ctx, b, dQ, dK, dV)
        fstep.find_sinks(ctx, b, dQ, dK, b.lse)
        fstep.sparse_layer(ctx, b, dQ, dK, dV, Kbar=Kbar)
        # the model's output for this step is synthetic: the AR(1) confidence of every gen position and a token id
        tok = (1000 + step * s.N + np.arange(s.N)).astype(np.int32)
        fb.focus_commit_step(ctx, torch.from_numpy(c_cur).cuda(), torch.from_numpy(tok).cuda(), s.M, None, None, s.N,
                             s.L, s.M, s.L, 2, d_conf, d_masked, d_x, picked, n_picked)
        torch.cuda.synchronize()
        S = oracle_sinks_by_head(t["Q"][active - s.M], t["K"], s.dtype, scale)
        sinks = fo.find_sinks(S, w.n_sink, 0, s.M)
        band = check_topk_band(b.sink_idx.cpu().numpy(), sinks, S, range(s.M), BAND, what=f"sinks step {step}")
        log_band(w.name, "sinks", f"step {step}", -1, band, w.n_sink, s.M)
        check_sinks_exact_on_own_scores(b.sink_idx.cpu().numpy(), fstep.from_device(b.sink_scores), w.n_sink, s.M,
                                        f"{w.name} step {step}")
        bi = b.block_idx.cpu().numpy().reshape(b.G, b.max_blocks)
        keep = b.sink_keep.cpu().numpy().reshape(b.G, -1)[:, :w.n_sink]
        check_block_sets(w, t, bi, keep, b.sink_idx.cpu().numpy(), focus, w.name, f"step {step}")
        if step in (0, 7, 15):
            check_layer(w, t, bi, keep, b.sink_idx.cpu().numpy(), focus, active, fstep.from_device(b.O),
                        fstep.from_device(b.lse), [0, 6, 13, 27], active)
        o_conf, o_masked, o_x, unmasked = fo.commit_step(o_conf, o_masked, o_x, gen_pos, c_cur, tok, s.M, s.L, 2)
        assert n_picked.item() == 2 and picked.cpu().numpy().tolist() == unmasked
        hits += len(set(unmasked) & set(focus.tolist()))
        total += len(unmasked)
        c_cur = wl.ar1_next(w.seed, step, c_cur)
    assert np.array_equal(d_masked.cpu().numpy(), o_masked) and np.array_equal(d_x.cpu().numpy(), o_x)
    assert np.array_equal(d_conf.cpu().numpy(), o_conf.astype(np.float32))
    assert o_masked[s.M:].sum() == s.N - 2 * w.n_steps and (o_x[s.M:] != 0).sum() == 2 * w.n_steps
    assert hits / total > 0.5                          # indicator recall on this synthetic process (logged, loose)
    assert ctx.poll_status() == 0


# ---- config 4: sweep points (context x keep ratio), gen-region rows ---------------------------------------------
@pytest.mark.parametrize("rows", ["gen", "active"])
@pytest.mark.parametrize("keep_den", wl.SWEEP_KEEP_DEN)
@pytest.mark.parametrize("L", wl.SWEEP_L)
def test_config4_sweep_points(ctx, L, keep_den, rows):
    """Every point of the context x keep-ratio grid that the sweep times, in both row modes: between them they take
    the one-warpgroup kernel (I_active rows), the key-pair form and the two-tile form (gen rows), short and long
    block lists, with and without staged tile lists."""
    w = wl.config(4, L=L, keep_den=keep_den)
    heads = [0, 21] if L > 40000 else [0, 13, 31]
    single_layer_case(ctx, w, rows, heads=heads, check_dense=L <= 40000)


# ---- the paper's own hyper-parameters (block 64, half of the blocks kept) on the 32K shape, one layer ---------
@pytest.mark.parametrize("rows", ["active", "gen"])
def test_paper_hyperparameters_one_layer(ctx, rows):
    """Prompt block size 64 and sparsity ratio 0.5 ("Implementation details"): 504 pooled blocks per head (the radix
    Top-C path), 252 kept, paired two per 128-key tile by the attention kernel."""
    w = wl.config(5)
    single_layer_case(ctx, w, rows, heads=[0, 22], check_dense=False)


# ---- the generator exactly as the benchmark text states it (sink keys x8, queries NOT shifted) ---------------------
@pytest.mark.parametrize("rows", ["active", "gen"])
def test_config0_with_the_literal_generator(ctx, rows):
    """Config 0 with unshifted queries: the planted sinks then carry only a fraction of a percent more attention mass
    than an ordinary key and sit inside the near-threshold band, so their recovery is not asserted; every index set
    still obeys the band rule and the outputs the 1e-5 bound."""
    w = wl.config(0)
    single_layer_case(ctx, w, rows, heads=list(range(w.shape.H)), variant="lit")


# ---- sink selection at the full config-2 shape with scores spread over decades: the band is empty ------------------
def test_sink_set_is_exactly_the_oracles_when_nothing_sits_near_the_threshold(ctx):
    """Config-2 shape (32 heads, 32K keys, the I_active rows) with keys whose logit against every query carries a
    common per-key offset a_j ~ N(0, 3): the attention mass S_j is roughly log-normal, spreads over two decades in
    the top percent alone, and for this seed no other candidate lies within 1e-3 of the 322nd largest score (the
    nearest are 3e-3 above and 1e-2 below).  The band rule then has nothing to forgive: the GPU's sink set must be
    the oracle's, index for index."""
    w = wl.config(2)
    s = w.shape
    rng = np.random.default_rng(78)
    c_prev, _ = wl.gen_confidence(w.seed, s.N)
    conf, masked = wl.full_conf(s, c_prev), wl.gen_masked(w)
    u = rng.standard_normal(s.d).astype(np.float32)
    u /= np.linalg.norm(u)
    a = (rng.standard_normal(s.L) * 3.0).astype(np.float32)
    Qs = wl.to_storage(rng.standard_normal((s.N, s.H, s.d), dtype=np.float32) + 3.0 * u, s.dtype)
    Ks = wl.to_storage(rng.standard_normal((s.Hkv, s.L, s.d), dtype=np.float32) +
                       (a[:, None] * u[None, :] * (math.sqrt(s.d) / 3.0))[None], s.dtype)
    dQ, dK = fstep.to_device(Qs, s.dtype), fstep.to_device(Ks, s.dtype)
    b = fstep.StepBuffers(w, rows="active")
    focus, active = run_selection(ctx, w, b, conf, masked)
    fstep.find_sinks(ctx, b, dQ, dK, None)               # no dense pass here: the library computes the LSE itself
    torch.cuda.synchronize()
    S = oracle_sinks_by_head(Qs[active - s.M], Ks, s.dtype, 1.0 / math.sqrt(s.d))
    sinks = fo.find_sinks(S, w.n_sink, 0, s.M)
    got = b.sink_idx.cpu().numpy()
    band = check_topk_band(got, sinks, S, range(s.M), BAND, what="spread sinks")
    log_band("c2 shape, log-normal attention mass", "sinks", "one layer", -1, band, w.n_sink, s.M)
    top = np.sort(S[:s.M])[::-1]
    assert top[0] / top[w.n_sink] > 50.0                  # the scores do spread
    assert band == 1                                      # the threshold element itself and nothing else
    assert got.tolist() == sinks.tolist()
    S_gpu = fstep.from_device(b.sink_scores)
    big = S[:s.M] >= top[w.n_sink] * 0.1                  # relative error where the mass is
    assert np.max(np.abs(S_gpu[:s.M][big] - S[:s.M][big]) / S[:s.M][big]) < 2e-3
    assert ctx.poll_status() == 0


# ---- Dream-7B's layer schedule: the last four layers stay dense ---------------------------------------------------
def test_dream_schedule_keeps_the_final_four_layers_dense(ctx):
    """Config-3 shape, 28 layers, layer_schedule(28, probe 5, final_dense 4) (the paper keeps the last four layers of
    Dream-7B dense): layers 0..5 dense (5 = probe), 6..23 sparse with the shared sink set, 24..27 dense again.  Per-layer
    Q/K/V seeded by the layer index; sampled layers of every kind are checked against the oracle, block sets of every
    group of the sampled sparse layers included."""
    w = wl.config(3)
    s = w.shape
    NL, probe = 28, 5
    sched = fstep.layer_schedule(NL, probe, final_dense=4)
    assert sched.count("sparse") == 18 and sched[24:] == ["dense"] * 4 and sched[probe] == "probe"
    check = {0: [0], probe: [13], 6: [0, 27], 23: [6], 24: [20], 27: [27]}
    c_prev, _ = wl.gen_confidence(w.seed, s.N)
    conf, masked = wl.full_conf(s, c_prev), wl.gen_masked(w)
    b = fstep.StepBuffers(w, rows="active")
    focus, active = run_selection(ctx, w, b, conf, masked)
    Kbar = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
    scale = 1.0 / math.sqrt(s.d)
    sinks_gpu = None
    for l, kind in enumerate(sched):
        t = wl.gen_qkv(s, 100 + l)
        dQ, dK, dV = (fstep.to_device(t[n], s.dtype) for n in "QKV")
        if kind in ("dense", "probe"):
            fstep.dense_layer(ctx, b, dQ, dK, dV)
            if kind == "probe":
                fstep.find_sinks(ctx, b, dQ, dK, b.lse)
                S = oracle_sinks_by_head(t["Q"][active - s.M], t["K"], s.dtype, scale)
                sinks = fo.find_sinks(S, w.n_sink, 0, s.M)
                band = check_topk_band(b.sink_idx.cpu().numpy(), sinks, S, range(s.M), BAND, what="sinks")
                log_band("dream schedule", "sinks", f"layer {l}", -1, band, w.n_sink, s.M)
                sinks_gpu = b.sink_idx.cpu().numpy()
        else:
            fb.focus_pool_keys(ctx, b.shape, dK, Kbar)
            fstep.sparse_layer(ctx, b, dQ, dK, dV, Kbar=Kbar)
        if l in check:
            torch.cuda.synchronize()
            bi = b.block_idx.cpu().numpy().reshape(b.G, b.max_blocks)
            keep = b.sink_keep.cpu().numpy().reshape(b.G, -1)[:, :w.n_sink]
            if kind == "sparse":
                check_block_sets(w, t, bi, keep, sinks_gpu, focus, "dream schedule", f"layer {l}")
            check_layer(w, t, bi, keep, sinks_gpu, focus, active, fstep.from_device(b.O), fstep.from_device(b.lse),
                        check[l], active, dense=kind != "sparse")
    assert ctx.poll_status() == 0
