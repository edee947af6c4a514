"""Seeded synthetic inputs for the Focus-dLLM hot path (shared by tests, smoke and bench).

This module holds input generation only: random Q/K/V with planted attention
sinks, confidence vectors, mask states and the hyper-parameters of the five
benchmark configurations.  It contains none of the method's arithmetic (no
top-k, no softmax, no pooling); the CUDA path and the CPU oracle both read the
arrays produced here and never each other's results.

Workload shapes follow the paper's efficiency study (context 8K-32K, generation
length 256-512, decoding block 32; Section "Experiments", "Implementation
details" and Appendix "Generation Settings") with LLaDA-8B (32 heads MHA,
head_dim 128) and Dream-7B (28 query / 4 KV heads) attention shapes.  The
paper's LongBench items and model weights are not available, so iid Gaussian
Q/K/V with planted sinks stand in for them.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional, Tuple

import numpy as np

SINK_NORM = 8.0          # planted sink keys get 8x the norm of a typical key
_TAG = {"q": 1, "k": 2, "v": 3, "u": 4, "sinkpos": 5, "conf": 6, "noise": 7, "mask": 8, "ar1": 9}


# ----------------------------------------------------------------------------
# bf16 storage helpers (storage format only: round-to-nearest-even and widening)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to the float32 values they denote (exact)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_storage(x32: np.ndarray, dtype: str) -> np.ndarray:
    """float32 -> storage array: float32 for 'f32', uint16 bit patterns for 'bf16'."""
    if dtype == "f32":
        return np.ascontiguousarray(x32, dtype=np.float32)
    if dtype == "bf16":
        return f32_to_bf16_bits(x32)
    raise ValueError(dtype)


def storage_to_f64(a: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of a storage array to float64 (what the oracle consumes)."""
    if dtype == "f32":
        return a.astype(np.float64)
    return bf16_bits_to_f32(a).astype(np.float64)


# ----------------------------------------------------------------------------
# shapes and configurations
# ----------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Shape:
    L: int            # total positions
    M: int            # prompt length; response/gen region is [M, L)
    H: int            # query heads
    Hkv: int          # key/value heads
    d: int            # head dim
    B: int            # prompt KV block size
    dtype: str        # 'f32' | 'bf16'

    @property
    def N(self) -> int:
        return self.L - self.M

    @property
    def nb(self) -> int:
        return (self.M + self.B - 1) // self.B


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    shape: Shape
    k: int                    # focus count (rounded rho * n)
    w: int                    # window size
    n_sink: int               # number of sink tokens, floor(M / 100)
    C: int                    # kept prompt blocks per group
    blk_lo: int               # current decoding block [blk_lo, blk_hi)
    blk_hi: int
    n_layers: int = 1
    probe_layer: int = 0      # 0-indexed layer whose attention identifies sinks
    n_steps: int = 1
    masked_count: Optional[int] = None   # c0: how many gen positions are still masked
    seed: int = 0


def config(idx: int, *, L: Optional[int] = None, keep_den: Optional[int] = None) -> Workload:
    """The five benchmark configurations (idx 0..4; idx 4, the sweep, takes L and keep_den = 1 / keep ratio) and,
    as idx 5, the paper's own hyper-parameters on the 32K shape."""
    if idx == 0:
        s = Shape(1024, 896, 8, 8, 64, 64, "f32")
        return Workload("c0_tiny_f32", s, k=16, w=8, n_sink=8, C=4, blk_lo=896, blk_hi=1024, masked_count=64)
    if idx == 1:
        s = Shape(8192, 7936, 32, 32, 128, 128, "bf16")
        return Workload("c1_llada_8k", s, k=8, w=8, n_sink=79, C=s.nb // 8, blk_lo=7936, blk_hi=7936 + 32)
    if idx == 2:
        s = Shape(32768, 32256, 32, 32, 128, 128, "bf16")
        return Workload("c2_llada_32k_32layers", s, k=8, w=8, n_sink=322, C=s.nb // 16, blk_lo=32256,
                        blk_hi=32256 + 32, n_layers=32, probe_layer=16)
    if idx == 3:
        s = Shape(16384, 16128, 28, 4, 128, 128, "bf16")
        return Workload("c3_dream_gqa_16k", s, k=8, w=8, n_sink=161, C=s.nb // 8, blk_lo=16128, blk_hi=16384,
                        n_steps=16)
    if idx == 5:
        # not one of the five benchmark configurations: the hyper-parameters of the paper's own experiments
        # (Implementation details: prompt block size 64, sparsity ratio 0.5, six dense layers, rho = 4, w = 8,
        # N_sink = 0.01 M) on the LLaDA attention shape at 32K context
        s = Shape(32768, 32256, 32, 32, 128, 64, "bf16")
        return Workload("c5_paper_hparams_32k", s, k=8, w=8, n_sink=322, C=s.nb // 2, blk_lo=32256,
                        blk_hi=32256 + 32, n_layers=32, probe_layer=5)
    if idx == 4:
        L = 32768 if L is None else L
        keep_den = 16 if keep_den is None else keep_den
        s = Shape(L, L - 256, 32, 32, 128, 128, "bf16")
        return Workload(f"c4_sweep_L{L}_keep1_{keep_den}", s, k=8, w=8, n_sink=s.M // 100, C=s.nb // keep_den,
                        blk_lo=s.M, blk_hi=s.M + 32)
    raise ValueError(idx)


SWEEP_L = [4096, 8192, 16384, 32768, 65536, 131072]
SWEEP_KEEP_DEN = [1, 4, 8, 16, 32]


# ----------------------------------------------------------------------------
# generators
# ----------------------------------------------------------------------------
def _rng(seed: int, tag: str, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), _TAG[tag], int(sub)])))


def sink_positions(seed: int, M: int) -> np.ndarray:
    """Planted sink positions: 0 and one seeded uniform position in [1, M)."""
    p = int(_rng(seed, "sinkpos").integers(1, M))
    return np.array([0, p], dtype=np.int64)


def sink_directions(seed: int, Hkv: int, d: int) -> np.ndarray:
    """One unit vector per KV head; both planted sinks of a head share it."""
    u = _rng(seed, "u").standard_normal((Hkv, d))
    return (u / np.linalg.norm(u, axis=1, keepdims=True)).astype(np.float32)


def gen_qkv(shape: Shape, seed: int, variant: str = "fix", threads: int = 0) -> Dict[str, np.ndarray]:
    """Q [N,H,d] for the gen-region positions M..L-1, K and V [Hkv,L,d], in storage dtype.

    Values are iid N(0,1)/sqrt(d).  Keys at the planted sink positions are
    replaced by SINK_NORM * u_g.  variant 'lit' stops there; variant 'fix'
    additionally adds u_{g(h)} to every query row so that the sink logit has a
    positive mean (8/sqrt(d)) and planted sinks carry about twice the attention
    mass of an ordinary key instead of a fraction of a percent more.
    """
    L, M, H, Hkv, d = shape.L, shape.M, shape.H, shape.Hkv, shape.d
    N = L - M
    inv = np.float32(1.0 / np.sqrt(d))
    u = sink_directions(seed, Hkv, d)
    spos = sink_positions(seed, M)
    sd = np.float32 if shape.dtype == "f32" else np.uint16
    K = np.empty((Hkv, L, d), dtype=sd)
    V = np.empty((Hkv, L, d), dtype=sd)

    def fill(job):
        tag, g = job
        x = _rng(seed, tag, g).standard_normal((L, d), dtype=np.float32) * inv
        if tag == "k":
            x[spos] = SINK_NORM * u[g]
            K[g] = to_storage(x, shape.dtype)
        else:
            V[g] = to_storage(x, shape.dtype)

    jobs = [(t, g) for g in range(Hkv) for t in ("k", "v")]
    if threads == 0:
        import os
        threads = min(32, os.cpu_count() or 1)
    if threads > 1 and len(jobs) > 1:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(fill, jobs))
    else:
        for j in jobs:
            fill(j)

    q = _rng(seed, "q").standard_normal((N, H, d), dtype=np.float32) * inv
    if variant == "fix":
        hpg = H // Hkv
        q = q + np.repeat(u, hpg, axis=0)[None, :, :]
    elif variant != "lit":
        raise ValueError(variant)
    return {"Q": to_storage(q, shape.dtype), "K": K, "V": V, "sink_pos": spos, "u": u}


def gen_confidence(seed: int, N: int, step: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """(c_prev, c_cur) over the N gen positions: Beta(2,5), then + N(0, 0.05) clipped to [0,1]."""
    c_prev = _rng(seed, "conf", step).beta(2.0, 5.0, size=N).astype(np.float32)
    noise = _rng(seed, "noise", step).normal(0.0, 0.05, size=N).astype(np.float32)
    c_cur = np.clip(c_prev + noise, 0.0, 1.0).astype(np.float32)
    return c_prev, c_cur


def gen_masked(wl: Workload) -> np.ndarray:
    """uint8[L] mask state at the (first) step: 1 = still [MASK]."""
    s = wl.shape
    m = np.zeros(s.L, dtype=np.uint8)
    if wl.masked_count is not None:
        pick = _rng(wl.seed, "mask").choice(s.N, size=wl.masked_count, replace=False)
        m[s.M + pick] = 1
    else:
        m[s.M:] = 1            # every gen position is still masked
    return m


def full_conf(shape: Shape, c_gen: np.ndarray) -> np.ndarray:
    """Embed per-gen-position confidences into a float32[L] vector (prompt entries 0)."""
    c = np.zeros(shape.L, dtype=np.float32)
    c[shape.M:] = c_gen
    return c


# AR(1) confidence process of the 16-step GQA configuration: stationary mean and
# standard deviation are those of Beta(2,5); correlation 0.9 between steps.
AR1_MU = 2.0 / 7.0
AR1_SD = float(np.sqrt(2.0 * 5.0 / (7.0 ** 2 * 8.0)))
AR1_RHO = 0.9


def ar1_next(seed: int, step: int, c: np.ndarray) -> np.ndarray:
    eps = _rng(seed, "ar1", step).standard_normal(c.shape[0]).astype(np.float32)
    nxt = AR1_MU + AR1_RHO * (c - AR1_MU) + np.sqrt(1.0 - AR1_RHO ** 2) * AR1_SD * eps
    return np.clip(nxt, 0.0, 1.0).astype(np.float32)


def unmask_two(masked: np.ndarray, conf: np.ndarray, lo: int, hi: int, n: int = 2) -> List[int]:
    """Harness-side stand-in for the transfer scheduler: clear the n masked positions in
    [lo, hi) with the highest current confidence (ties: lower index).  Mutates `masked`."""
    cand = [i for i in range(lo, hi) if masked[i]]
    cand.sort(key=lambda i: (-float(conf[i]), i))
    out = cand[:n]
    for i in out:
        masked[i] = 0
    return out
