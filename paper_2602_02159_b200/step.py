"""Device-buffer bookkeeping for one Focus-dLLM denoising step (harness level).

`StepBuffers` owns the caller-side buffers the C ABI writes into (index sets, counts, block scores, outputs)
and `run_layer_*` issue the library calls of one layer in the order of Algorithm 1.  No arithmetic happens
here; torch tensors are device memory only.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np
import torch

from . import binding as fb
from .workloads import Shape, Workload


def torch_dtype(dtype: str):
    return torch.float32 if dtype == "f32" else torch.bfloat16


def to_device(a: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    """Storage array (float32, or uint16 bf16 bit patterns) -> device tensor of the matching torch dtype."""
    if dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(a)).to(device)
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def from_device(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> float64 numpy (exact widening)."""
    return t.detach().to(torch.float64).cpu().numpy()


def c_shape(s: Shape) -> fb.focus_shape:
    return fb.make_shape(s.L, s.M, s.H, s.Hkv, s.d, s.B, fb.F32 if s.dtype == "f32" else fb.BF16)


@dataclasses.dataclass
class StepBuffers:
    """Caller-owned outputs of the selection stages and of attention for one workload."""
    wl: Workload
    head_reduce: int = fb.HEADS_PER_KV_GROUP
    sink_mode: int = fb.SINK_TOKENS
    # "active": attention rows are I_active (the paper), Q holds every gen row; "gen": all N gen rows are attention rows;
    # "compact": attention rows are I_active and Q holds ONLY those rows, in list order (a caller that computed or
    # uploaded nothing else): row r of Q belongs to position active_idx[r]
    rows: str = "active"
    device: str = "cuda"

    def __post_init__(self):
        w, s = self.wl, self.wl.shape
        dev = self.device
        i32 = dict(dtype=torch.int32, device=dev)
        self.shape = c_shape(s)
        self.max_active = max(1, w.k * (2 * (w.w // 2) + 1))
        self.G = 1 if self.head_reduce == fb.HEADS_ALL else s.Hkv
        self.max_blocks = max(1, min(s.nb, w.C + w.n_sink) if self.sink_mode == fb.SINK_BLOCKS else w.C)
        self.focus_idx = torch.full((max(1, w.k),), -1, **i32)
        self.n_focus = torch.zeros(1, **i32)
        self.active_idx = torch.full((self.max_active,), -1, **i32)
        self.n_active = torch.zeros(1, **i32)
        self.sink_idx = torch.full((max(1, w.n_sink),), -1, **i32)
        self.sink_scores = torch.zeros(s.L, dtype=torch.float32, device=dev)
        self.R = torch.zeros(self.G * max(1, s.nb), dtype=torch.float32, device=dev)
        self.block_idx = torch.full((self.G * self.max_blocks,), -1, **i32)
        self.block_cnt = torch.zeros(self.G, **i32)
        self.sink_keep = torch.zeros(self.G * max(1, w.n_sink), dtype=torch.uint8, device=dev)
        self.max_rows = s.N if self.rows == "gen" else self.max_active
        self.O = torch.zeros(self.max_rows, s.H, s.d, dtype=torch_dtype(s.dtype), device=dev)
        self.lse = torch.zeros(s.H, self.max_rows, dtype=torch.float32, device=dev)
        # compact mode: Q row r <-> active_idx[r]; the library is handed local row numbers
        self.row_ids = torch.arange(self.max_active, **i32)
        self.focus_local = torch.full((max(1, w.k),), -1, **i32)
        self.q_base = 0 if self.rows == "compact" else s.M
        self.n_q = self.max_active if self.rows == "compact" else s.N

    # rows argument triple of the attention calls
    def _rows(self):
        if self.rows == "active":
            return self.active_idx, self.n_active, self.max_active
        if self.rows == "compact":
            return self.row_ids, self.n_active, self.max_active
        return None, None, 0

    def _focus(self):
        return self.focus_local if self.rows == "compact" else self.focus_idx

    def set_local_focus(self, focus_pos, active_pos):
        """Compact mode: where each focus position sits in the active list (index bookkeeping on the host, after the
        caller has read the two lists back to gather its query rows)."""
        where = {int(p): r for r, p in enumerate(active_pos)}
        loc = [where[int(p)] for p in focus_pos]
        self.focus_local[:len(loc)].copy_(torch.tensor(loc, dtype=torch.int32), non_blocking=True)


def select_queries(ctx, b: StepBuffers, conf_prev: torch.Tensor, masked: torch.Tensor, stream=None):
    w, s = b.wl, b.wl.shape
    fb.focus_select_queries(ctx, conf_prev, masked, s.L, w.blk_lo, w.blk_hi, w.k, w.w, s.M, s.L,
                            b.focus_idx, b.n_focus, b.active_idx, b.n_active, stream)


def dense_layer(ctx, b: StepBuffers, Q, K, V, O=None, lse=None, stream=None):
    s = b.wl.shape
    q_rows, n_rows, max_rows = b._rows()
    fb.focus_dense_attn(ctx, b.shape, Q, b.q_base, b.n_q, q_rows, n_rows, max_rows, K, V, b.O if O is None else O,
                        b.lse if lse is None else lse, stream)


def find_sinks(ctx, b: StepBuffers, Q, K, lse: Optional[torch.Tensor], stream=None):
    """lse must be the [H, max_active] log-sum-exp of a dense pass over the I_active rows, or None."""
    w, s = b.wl, b.wl.shape
    act = b.row_ids if b.rows == "compact" else b.active_idx
    fb.focus_find_sinks(ctx, b.shape, Q, b.q_base, act, b.n_active, b.max_active, K, lse, w.n_sink, 0, s.M,
                        b.sink_idx, b.sink_scores, stream)


def find_sinks_sharded(ctx, b: StepBuffers, Q, K, lse: Optional[torch.Tensor], group=None, stream=None):
    """find_sinks for a rank that holds only its own heads of the layer (b.shape, Q, K and lse describe those heads):
    S over the local heads, mean over the ranks of `group` (the one exchange of a step), Top-N_sink from the mean.
    Every rank ends up with the same b.sink_idx and b.sink_scores."""
    from . import head_shards
    w, s = b.wl, b.wl.shape
    act = b.row_ids if b.rows == "compact" else b.active_idx
    fb.focus_find_sinks(ctx, b.shape, Q, b.q_base, act, b.n_active, b.max_active, K, lse, 0, 0, s.M, None,
                        b.sink_scores, stream)
    head_shards.mean_over_ranks(b.sink_scores, group)
    fb.focus_select_sinks(ctx, b.sink_scores, s.L, 0, s.M, w.n_sink, b.sink_idx, stream)


def sparse_layer(ctx, b: StepBuffers, Q, K, V, Kbar: Optional[torch.Tensor] = None, O=None, lse=None, stream=None,
                 fused: bool = True):
    """score_blocks -> select_blocks -> sparse_attn for one sparse layer (Algorithm 1, sparse branch); with cached
    pooled keys and the default modes this is the single fused call focus_sparse_layer."""
    w, s = b.wl, b.wl.shape
    q_rows, n_rows, max_rows = b._rows()
    if Kbar is not None and b.head_reduce == fb.HEADS_PER_KV_GROUP and b.sink_mode == fb.SINK_TOKENS and fused:
        fb.focus_sparse_layer(ctx, b.shape, Q, b.q_base, b.n_q, q_rows, n_rows, max_rows, b._focus(), b.n_focus, max(1, w.k),
                              K, V, Kbar, w.C, b.sink_idx, w.n_sink, b.R, b.block_idx, b.block_cnt, b.sink_keep,
                              b.O if O is None else O, b.lse if lse is None else lse, stream)
        return
    fb.focus_score_blocks(ctx, b.shape, Q, b.q_base, b._focus(), b.n_focus, max(1, w.k), None if Kbar is not None else K,
                          Kbar, b.head_reduce, b.R, stream)
    fb.focus_select_blocks(ctx, b.shape, b.R, b.head_reduce, w.C, b.sink_idx, w.n_sink, b.sink_mode, b.block_idx,
                           b.max_blocks, b.block_cnt, b.sink_keep, stream)
    fb.focus_sparse_attn(ctx, b.shape, Q, b.q_base, b.n_q, q_rows, n_rows, max_rows, K, V, b.head_reduce, b.block_idx,
                         b.max_blocks, b.block_cnt, b.sink_idx, b.sink_keep, w.n_sink, b.O if O is None else O,
                         b.lse if lse is None else lse, stream)


def layer_schedule(n_layers: int, probe_layer: int, final_dense: int = 0):
    """Which attention each layer of a non-block-entry step runs: 'dense' for layers 0..probe_layer (the probe layer
    also identifies the sinks), 'sparse' after it, except that the last `final_dense` layers stay dense (the paper
    keeps the final four layers of Dream-7B dense; 0 for UltraLLaDA)."""
    out = []
    for l in range(n_layers):
        if l <= probe_layer or l >= n_layers - final_dense:
            out.append("probe" if l == probe_layer else "dense")
        else:
            out.append("sparse")
    return out
