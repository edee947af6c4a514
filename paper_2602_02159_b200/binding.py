"""ctypes binding of libfocus.so: same names as include/focus.h, argument marshalling only.

Tensors are torch CUDA tensors used purely as device buffers; every step of the path runs inside the
library's kernels.  There is no fallback: if libfocus.so is missing or a call fails, this raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("FOCUS_LIB_PATH") or os.path.join(HERE, "libfocus.so")   # override: an alternative build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1
HEADS_PER_KV_GROUP, HEADS_ALL = 0, 1
SINK_TOKENS, SINK_BLOCKS = 0, 1
OPT_MERGE_MODE, OPT_NO_WIDE, OPT_NO_PDL = 0, 1, 2
MERGE_AUTO, MERGE_COUNTERS, MERGE_KERNEL = 0, 1, 2


class FocusError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (focus_status {code})")


class focus_shape(C.Structure):
    _fields_ = [("L", C.c_int32), ("M", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("kv_block", C.c_int32), ("dtype", C.c_int32),
                ("softmax_scale", C.c_float), ("q_stride_row", C.c_int64), ("q_stride_head", C.c_int64),
                ("kv_stride_tok", C.c_int64), ("kv_stride_head", C.c_int64)]


_lib = None
_P, _I, _Z = C.c_void_p, C.c_int32, C.c_size_t
_SH = C.POINTER(focus_shape)

_SIGS = {
    "focus_create": (_I, [C.POINTER(_P), C.c_int, _Z]),
    "focus_destroy": (_I, [_P]),
    "focus_workspace_bytes": (_I, [_SH, _I, _I, _I, C.POINTER(_Z)]),
    "focus_poll_status": (_I, [_P, _P, C.POINTER(_I)]),
    "focus_status_string": (C.c_char_p, [_I]),
    "focus_set_force_simt": (_I, [_P, _I]),
    "focus_set_option": (_I, [_P, _I, _I]),
    "focus_selftest_bounded_wait": (_I, [_P, _I, _P]),
    "focus_stream_read": (_I, [_P, _P, _Z, _P, _P]),
    "focus_launch_count": (C.c_uint64, []),
    "focus_last_attn_variant": (_I, [_P]),
    "focus_select_queries": (_I, [_P, _P, _P, _I, _I, _I, _I, _I, _I, _I, _P, _P, _P, _P, _P]),
    "focus_find_sinks": (_I, [_P, _SH, _P, _I, _P, _P, _I, _P, _P, _I, _I, _I, _P, _P, _P]),
    "focus_select_sinks": (_I, [_P, _P, _I, _I, _I, _I, _P, _P]),
    "focus_pool_keys": (_I, [_P, _SH, _P, _P, _P]),
    "focus_score_blocks": (_I, [_P, _SH, _P, _I, _P, _P, _I, _P, _P, _I, _P, _P]),
    "focus_score_blocks_static": (_I, [_SH, _P, _I, _P, _P, _I, _P, _P, _I, _P, _P, _P]),
    "focus_select_blocks": (_I, [_P, _SH, _P, _I, _I, _P, _I, _I, _P, _I, _P, _P, _P]),
    "focus_sparse_attn": (_I, [_P, _SH, _P, _I, _I, _P, _P, _I, _P, _P, _I, _P, _I, _P, _P, _P, _I, _P, _P, _P]),
    "focus_sparse_layer": (_I, [_P, _SH, _P, _I, _I, _P, _P, _I, _P, _P, _I, _P, _P, _P, _I, _P, _I, _P, _P, _P, _P, _P,
                                _P, _P]),
    "focus_confidence": (_I, [_P, _P, _I, C.c_int64, _I, _I, _I, _P, _P, _I, _P, _P, _P]),
    "focus_update_kv": (_I, [_P, _SH, _P, _P, _P, _P, _P, _P, _I, _P]),
    "focus_update_pooled_keys": (_I, [_P, _SH, _P, _P, _P, _P, _I, _P]),
    "focus_commit_step": (_I, [_P, _P, _P, _I, _P, _P, _I, _I, _I, _I, _I, _P, _P, _P, _P, _P, _P]),
    "focus_dense_attn": (_I, [_P, _SH, _P, _I, _I, _P, _P, _I, _P, _P, _P, _P, _P]),
}


def load_library(path: Optional[str] = None):
    """dlopen libfocus.so and set the prototypes.  Raises if the library has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} is missing: build it with `python -m paper_2602_02159_b200.build` "
                                "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(p)
    for name, (res, args) in _SIGS.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    if path is None:
        _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().focus_status_string(code).decode()


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(code: int, where: str):
    if code != OK:
        raise FocusError(code, where)


def make_shape(L, M, H, Hkv, d, B, dtype, q_stride_row=None, q_stride_head=None, kv_stride_tok=None,
               kv_stride_head=None, softmax_scale=0.0) -> focus_shape:
    """Strides default to contiguous Q [rows, H, d] and K/V [Hkv, L, d]."""
    return focus_shape(L, M, H, Hkv, d, B, dtype, softmax_scale,
                       H * d if q_stride_row is None else q_stride_row,
                       d if q_stride_head is None else q_stride_head,
                       d if kv_stride_tok is None else kv_stride_tok,
                       L * d if kv_stride_head is None else kv_stride_head)


class Context:
    """Owns a focus_ctx (device, workspace, status word)."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self._lib = load_library()
        h = _P()
        _check(self._lib.focus_create(C.byref(h), device, workspace_bytes), "focus_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            self._lib.focus_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def poll_status(self, stream=None) -> int:
        v = _I(0)
        _check(self._lib.focus_poll_status(self.handle, _stream(stream), C.byref(v)), "focus_poll_status")
        return v.value

    def last_attn_variant(self) -> int:
        return self._lib.focus_last_attn_variant(self.handle)

    def set_force_simt(self, force: bool) -> int:
        return self._lib.focus_set_force_simt(self.handle, 1 if force else 0)

    def set_option(self, option: int, value: int) -> int:
        """focus_set_option: returns the previous value; raises on a bad option or value."""
        prev = self._lib.focus_set_option(self.handle, int(option), int(value))
        if prev < 0:
            raise FocusError(ERR_INVALID_ARG, "focus_set_option")
        return prev

    def selftest_bounded_wait(self, limit_us: int, stream=None) -> None:
        """One small CTA waits limit_us microseconds on a barrier nobody arrives at, then gives up: poll_status()
        reports ERR_TIMEOUT afterwards."""
        _check(self._lib.focus_selftest_bounded_wait(self.handle, int(limit_us), _stream(stream)),
               "focus_selftest_bounded_wait")


def focus_stream_read(ctx, buf, nbytes, checksum, stream=None):
    """Read-only pass over nbytes of `buf`; the xor of its 32-bit words lands in checksum[0] (uint32 / int32 tensor)."""
    _check(ctx._lib.focus_stream_read(ctx.handle, _ptr(buf), int(nbytes), _ptr(checksum), _stream(stream)),
           "focus_stream_read")


def focus_launch_count() -> int:
    return int(load_library().focus_launch_count())


def focus_workspace_bytes(shape: focus_shape, n_q: int, max_blocks: int, n_sink: int) -> int:
    out = _Z(0)
    _check(load_library().focus_workspace_bytes(C.byref(shape), n_q, max_blocks, n_sink, C.byref(out)),
           "focus_workspace_bytes")
    return out.value


def focus_select_queries(ctx, conf_prev, masked, L, blk_lo, blk_hi, k, w, clip_lo, clip_hi,
                         focus_idx, n_focus, active_idx, n_active, stream=None):
    _check(ctx._lib.focus_select_queries(ctx.handle, _ptr(conf_prev), _ptr(masked), L, blk_lo, blk_hi, k, w, clip_lo,
                                         clip_hi, _ptr(focus_idx), _ptr(n_focus), _ptr(active_idx), _ptr(n_active),
                                         _stream(stream)), "focus_select_queries")


def focus_find_sinks(ctx, shape, Q, q_base, active_idx, n_active, max_active, K, lse, n_sink, cand_lo, cand_hi,
                     sink_idx, scores=None, stream=None):
    _check(ctx._lib.focus_find_sinks(ctx.handle, C.byref(shape), _ptr(Q), q_base, _ptr(active_idx), _ptr(n_active),
                                     max_active, _ptr(K), _ptr(lse), n_sink, cand_lo, cand_hi, _ptr(sink_idx),
                                     _ptr(scores), _stream(stream)), "focus_find_sinks")


def focus_select_sinks(ctx, scores, L, cand_lo, cand_hi, n_sink, sink_idx, stream=None):
    _check(ctx._lib.focus_select_sinks(ctx.handle, _ptr(scores), L, cand_lo, cand_hi, n_sink, _ptr(sink_idx),
                                       _stream(stream)), "focus_select_sinks")


def focus_pool_keys(ctx, shape, K, Kbar, stream=None):
    _check(ctx._lib.focus_pool_keys(ctx.handle, C.byref(shape), _ptr(K), _ptr(Kbar), _stream(stream)),
           "focus_pool_keys")


def focus_score_blocks(ctx, shape, Q, q_base, focus_idx, n_focus, max_focus, K, Kbar, head_reduce, R, stream=None):
    _check(ctx._lib.focus_score_blocks(ctx.handle, C.byref(shape), _ptr(Q), q_base, _ptr(focus_idx), _ptr(n_focus),
                                       max_focus, _ptr(K), _ptr(Kbar), head_reduce, _ptr(R), _stream(stream)),
           "focus_score_blocks")


def focus_score_blocks_static(shape, Q, q_base, focus_idx, n_focus, max_focus, K, Kbar, head_reduce, R,
                              device_status=None, stream=None):
    """Block relevance (Eq. 7) without a context and without any allocation: for callers that live inside someone
    else's memory budget.  Scratch is a fixed array inside the library (limits in include/focus.h); calls that
    overlap on the GPU race on it, and the first call on a device should precede any stream capture."""
    _check(load_library().focus_score_blocks_static(C.byref(shape), _ptr(Q), q_base, _ptr(focus_idx), _ptr(n_focus),
                                                    max_focus, _ptr(K), _ptr(Kbar), head_reduce, _ptr(R),
                                                    _ptr(device_status), _stream(stream)),
           "focus_score_blocks_static")


def focus_select_blocks(ctx, shape, R, head_reduce, C_keep, sink_idx, n_sink, sink_mode, block_idx, max_blocks,
                        block_cnt, sink_keep, stream=None):
    _check(ctx._lib.focus_select_blocks(ctx.handle, C.byref(shape), _ptr(R), head_reduce, C_keep, _ptr(sink_idx),
                                        n_sink, sink_mode, _ptr(block_idx), max_blocks, _ptr(block_cnt),
                                        _ptr(sink_keep), _stream(stream)), "focus_select_blocks")


def focus_sparse_attn(ctx, shape, Q, q_base, n_q, q_rows, n_rows, max_rows, K, V, head_reduce, block_idx, max_blocks,
                      block_cnt, sink_idx, sink_keep, n_sink, O, lse=None, stream=None):
    _check(ctx._lib.focus_sparse_attn(ctx.handle, C.byref(shape), _ptr(Q), q_base, n_q, _ptr(q_rows), _ptr(n_rows),
                                      max_rows, _ptr(K), _ptr(V), head_reduce, _ptr(block_idx), max_blocks,
                                      _ptr(block_cnt), _ptr(sink_idx), _ptr(sink_keep), n_sink, _ptr(O), _ptr(lse),
                                      _stream(stream)), "focus_sparse_attn")


def focus_sparse_layer(ctx, shape, Q, q_base, n_q, q_rows, n_rows, max_rows, focus_idx, n_focus, max_focus, K, V, Kbar,
                       C_keep, sink_idx, n_sink, R, block_idx, block_cnt, sink_keep, O, lse=None, stream=None):
    _check(ctx._lib.focus_sparse_layer(ctx.handle, C.byref(shape), _ptr(Q), q_base, n_q, _ptr(q_rows), _ptr(n_rows),
                                       max_rows, _ptr(focus_idx), _ptr(n_focus), max_focus, _ptr(K), _ptr(V),
                                       _ptr(Kbar), C_keep, _ptr(sink_idx), n_sink, _ptr(R), _ptr(block_idx),
                                       _ptr(block_cnt), _ptr(sink_keep), _ptr(O), _ptr(lse), _stream(stream)),
           "focus_sparse_layer")


def focus_dense_attn(ctx, shape, Q, q_base, n_q, q_rows, n_rows, max_rows, K, V, O, lse=None, stream=None):
    _check(ctx._lib.focus_dense_attn(ctx.handle, C.byref(shape), _ptr(Q), q_base, n_q, _ptr(q_rows), _ptr(n_rows),
                                     max_rows, _ptr(K), _ptr(V), _ptr(O), _ptr(lse), _stream(stream)),
           "focus_dense_attn")


def focus_confidence(ctx, logits, dtype, row_stride, vocab, pos_base, n_pos, rows, n_rows, max_rows, conf, token,
                     stream=None):
    _check(ctx._lib.focus_confidence(ctx.handle, _ptr(logits), dtype, row_stride, vocab, pos_base, n_pos, _ptr(rows),
                                     _ptr(n_rows), max_rows, _ptr(conf), _ptr(token), _stream(stream)),
           "focus_confidence")


def focus_update_kv(ctx, shape, K_cache, V_cache, K_new, V_new, rows, n_rows, max_rows, stream=None):
    _check(ctx._lib.focus_update_kv(ctx.handle, C.byref(shape), _ptr(K_cache), _ptr(V_cache), _ptr(K_new), _ptr(V_new),
                                    _ptr(rows), _ptr(n_rows), max_rows, _stream(stream)), "focus_update_kv")


def focus_update_pooled_keys(ctx, shape, K, Kbar, rows, n_rows, max_rows, stream=None):
    _check(ctx._lib.focus_update_pooled_keys(ctx.handle, C.byref(shape), _ptr(K), _ptr(Kbar), _ptr(rows), _ptr(n_rows),
                                             max_rows, _stream(stream)), "focus_update_pooled_keys")


def focus_commit_step(ctx, conf_new, token_new, pos_base, rows, n_rows, max_rows, L, blk_lo, blk_hi, n_unmask, conf,
                      masked, x, unmasked_idx=None, n_unmasked=None, stream=None):
    _check(ctx._lib.focus_commit_step(ctx.handle, _ptr(conf_new), _ptr(token_new), pos_base, _ptr(rows), _ptr(n_rows),
                                      max_rows, L, blk_lo, blk_hi, n_unmask, _ptr(conf), _ptr(masked), _ptr(x),
                                      _ptr(unmasked_idx), _ptr(n_unmasked), _stream(stream)), "focus_commit_step")
