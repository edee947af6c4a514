// Context management, argument validation and dispatch of the attention and sink entry points.
#include <stdio.h>
#include <stdlib.h>

#include <new>

#include <string.h>

#include "focus_common.cuh"

focus_status launch_sink_select(focus_ctx* ctx, const float* part, int H, int L, const int32_t* n_active, float* S,
                                int cand_lo, int cand_hi, int n_sink, int32_t* sink_idx, cudaStream_t st);
focus_status launch_sink_topn(focus_ctx* ctx, const float* S, const int32_t* n_active, int cand_lo, int cand_hi,
                              int n_sink, int32_t* sink_idx, cudaStream_t st);
focus_status launch_sink_colsum_simt(focus_ctx* ctx, const focus_shape* s, const void* Q, int q_base,
                                     const int32_t* active_idx, const int32_t* n_active, int max_active,
                                     const void* K, const float* lse, float* part, cudaStream_t st);
bool sink_tc_supported(const focus_ctx* ctx, const focus_shape* s, int max_active);
focus_status launch_sink_colsum_tc(focus_ctx* ctx, const focus_shape* s, const void* Q, int q_base,
                                   const int32_t* active_idx, const int32_t* n_active, int max_active, const void* K,
                                   const float* lse, float* part, WsAlloc& ws, cudaStream_t st);

unsigned long long g_focus_launches = 0;

extern "C" uint64_t focus_launch_count(void) { return g_focus_launches; }

extern "C" const char* focus_status_string(focus_status s) {
  switch (s) {
    case FOCUS_OK: return "ok";
    case FOCUS_ERR_INVALID_ARG: return "invalid argument";
    case FOCUS_ERR_UNSUPPORTED: return "unsupported shape or mode";
    case FOCUS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case FOCUS_ERR_CUDA: return "CUDA error";
    case FOCUS_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" focus_status focus_create(focus_ctx** out, int device, size_t workspace_bytes) {
  if (!out) return FOCUS_ERR_INVALID_ARG;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return FOCUS_ERR_CUDA;
  if (cudaSetDevice(device) != cudaSuccess) return FOCUS_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FOCUS_ERR_CUDA;
  focus_ctx* c = new (std::nothrow) focus_ctx();
  if (!c) return FOCUS_ERR_CUDA;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->ws_bytes = workspace_bytes ? workspace_bytes : (size_t)256 << 20;
  c->force_simt = 0;
  c->last_attn_variant = 0;
  c->no_wide = 0;
  c->no_pdl = 0;
  c->merge_mode = 0;
  c->encode_tiled = nullptr;
  if (prop.major == 10) {   // tensor-core kernels are built for sm_100a only
    cudaDriverEntryPointQueryResult q;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      c->encode_tiled = fn;
  }
  if (cudaMalloc(&c->ws, c->ws_bytes) != cudaSuccess ||
      cudaMalloc(&c->d_status, 256 + FOCUS_N_COUNTERS * sizeof(int32_t)) != cudaSuccess) {
    if (c->ws) cudaFree(c->ws);
    delete c;
    return FOCUS_ERR_CUDA;
  }
  cudaMemset(c->d_status, 0, 256 + FOCUS_N_COUNTERS * sizeof(int32_t));
  c->d_counters = c->d_status + 64;
  *out = c;
  return FOCUS_OK;
}

extern "C" focus_status focus_destroy(focus_ctx* ctx) {
  if (!ctx) return FOCUS_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaFree(ctx->ws);
  cudaFree(ctx->d_status);
  delete ctx;
  return FOCUS_OK;
}

extern "C" int32_t focus_set_force_simt(focus_ctx* ctx, int32_t force) {
  if (!ctx) return -1;
  const int prev = ctx->force_simt;
  ctx->force_simt = force ? 1 : 0;
  return prev;
}

extern "C" int32_t focus_set_option(focus_ctx* ctx, int32_t option, int32_t value) {
  if (!ctx) return -1;
  int* slot = nullptr;
  int max_value = 1;
  switch (option) {
    case FOCUS_OPT_MERGE_MODE: slot = &ctx->merge_mode; max_value = 2; break;
    case FOCUS_OPT_NO_WIDE: slot = &ctx->no_wide; break;
    case FOCUS_OPT_NO_PDL: slot = &ctx->no_pdl; break;
    default: return -1;
  }
  if (value < 0 || value > max_value) return -1;
  const int prev = *slot;
  *slot = value;
  return prev;
}

extern "C" int32_t focus_last_attn_variant(focus_ctx* ctx) { return ctx ? ctx->last_attn_variant : -1; }

extern "C" focus_status focus_poll_status(focus_ctx* ctx, focus_stream stream, int32_t* device_status) {
  if (!ctx || !device_status) return FOCUS_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return FOCUS_ERR_CUDA;
  if (cudaMemcpy(device_status, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess)
    return FOCUS_ERR_CUDA;
  if (*device_status != 0 && cudaMemset(ctx->d_status, 0, sizeof(int32_t)) != cudaSuccess) return FOCUS_ERR_CUDA;
  return FOCUS_OK;
}

extern "C" focus_status focus_workspace_bytes(const focus_shape* shape, int32_t n_q, int32_t max_blocks,
                                              int32_t n_sink, size_t* out_bytes) {
  if (!shape_ok_basic(shape) || !out_bytes || n_q < 0 || max_blocks < 0 || n_sink < 0) return FOCUS_ERR_INVALID_ARG;
  const size_t H = shape->n_q_heads, L = shape->L;
  size_t sink = H * L * 4 + L * 4 + H * (size_t)n_q * 4 + (size_t)n_q * H * shape->head_dim * 2 + 4096;
  size_t score = (size_t)shape->n_kv_heads * (shape->head_dim + shape_nb(shape)) * 4 + 1024;
  size_t attn = attn_tc_workspace(shape, n_q, max_blocks, n_sink);
  // focus_find_sinks without a log-sum-exp runs an attention pass on top of its own buffers: the two add up
  size_t m = sink + attn;
  *out_bytes = (m > score ? m : score) + 4096;
  return FOCUS_OK;
}

// ---- attention dispatch ---------------------------------------------------------------------------
static focus_status attn_common(focus_ctx* ctx, const focus_shape* shape, const void* Q, int q_base, int n_q,
                                const int32_t* q_rows, const int32_t* n_rows, int max_rows, const void* K,
                                const void* V, void* O, float* lse, AttnArgs& a) {
  if (!ctx || !shape_ok_basic(shape) || !Q || !K || !V || !O) return FOCUS_ERR_INVALID_ARG;
  if (!all_aligned16(Q, K, V, O)) return FOCUS_ERR_INVALID_ARG;
  if (n_q < 0 || q_base < 0 || q_base + n_q > shape->L) return FOCUS_ERR_INVALID_ARG;
  if ((q_rows == nullptr) != (n_rows == nullptr)) return FOCUS_ERR_INVALID_ARG;
  if (q_rows && max_rows < 0) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;
  a.sh = *shape;
  a.scale = shape_scale(shape);
  a.Q = Q; a.q_base = q_base; a.n_q = n_q; a.q_rows = q_rows; a.n_rows = n_rows;
  a.max_rows = q_rows ? max_rows : n_q;
  a.K = K; a.V = V; a.O = O; a.lse = lse; a.lse_stride = a.max_rows;
  return FOCUS_OK;
}

static focus_status attn_dispatch(focus_ctx* ctx, const AttnArgs& a, cudaStream_t st) {
  if (a.max_rows == 0) return FOCUS_OK;
  if (!ctx->force_simt && attn_tc_supported(ctx, a)) return launch_attn_tc(ctx, a, st);
  ctx->last_attn_variant = 1;
  return launch_attn_simt(ctx, a, st);
}

extern "C" focus_status focus_dense_attn(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base,
                                         int32_t n_q, const int32_t* q_rows, const int32_t* n_rows, int32_t max_rows,
                                         const void* K, const void* V, void* O, float* lse, focus_stream stream) {
  FOCUS_STAGE("focus_dense_attn");
  AttnArgs a{};
  focus_status s = attn_common(ctx, shape, Q, q_base, n_q, q_rows, n_rows, max_rows, K, V, O, lse, a);
  if (s != FOCUS_OK) return s;
  a.dense = 1;
  return attn_dispatch(ctx, a, stream);
}

extern "C" focus_status focus_sparse_attn(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base,
                                          int32_t n_q, const int32_t* q_rows, const int32_t* n_rows, int32_t max_rows,
                                          const void* K, const void* V, int32_t head_reduce, const int32_t* block_idx,
                                          int32_t max_blocks, const int32_t* block_cnt, const int32_t* sink_idx,
                                          const uint8_t* sink_keep, int32_t n_sink, void* O, float* lse,
                                          focus_stream stream) {
  FOCUS_STAGE("focus_sparse_attn");
  AttnArgs a{};
  focus_status s = attn_common(ctx, shape, Q, q_base, n_q, q_rows, n_rows, max_rows, K, V, O, lse, a);
  if (s != FOCUS_OK) return s;
  if (head_reduce != FOCUS_HEADS_PER_KV_GROUP && head_reduce != FOCUS_HEADS_ALL) return FOCUS_ERR_INVALID_ARG;
  if (!block_idx || !block_cnt || max_blocks < 0 || n_sink < 0) return FOCUS_ERR_INVALID_ARG;
  if (n_sink > 0 && (!sink_idx || !sink_keep)) return FOCUS_ERR_INVALID_ARG;
  a.dense = 0;
  a.group_stride = head_reduce == FOCUS_HEADS_ALL ? 0 : 1;
  a.block_idx = block_idx; a.max_blocks = max_blocks; a.block_cnt = block_cnt;
  a.sink_idx = sink_idx; a.sink_keep = sink_keep; a.n_sink = n_sink;
  return attn_dispatch(ctx, a, stream);
}

// ---- sinks ---------------------------------------------------------------------------------------
extern "C" focus_status focus_find_sinks(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base,
                                         const int32_t* active_idx, const int32_t* n_active, int32_t max_active,
                                         const void* K, const float* lse, int32_t n_sink, int32_t cand_lo,
                                         int32_t cand_hi, int32_t* sink_idx, float* scores, focus_stream stream) {
  FOCUS_STAGE("focus_find_sinks");
  if (!ctx || !shape_ok_basic(shape) || !Q || !active_idx || !n_active || !K) return FOCUS_ERR_INVALID_ARG;
  if (n_sink > 0 && !sink_idx) return FOCUS_ERR_INVALID_ARG;      // n_sink == 0: scores only
  if (!all_aligned16(Q, K)) return FOCUS_ERR_INVALID_ARG;
  if (max_active <= 0 || n_sink < 0 || q_base < 0 || q_base > shape->L) return FOCUS_ERR_INVALID_ARG;
  if (cand_lo < 0 || cand_hi < cand_lo || cand_hi > shape->L) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;
  const int H = shape->n_q_heads, L = shape->L;
  WsAlloc ws(ctx);
  float* part = ws.get<float>((size_t)H * L);
  float* S = scores ? scores : ws.get<float>(L);
  float* lse_buf = lse ? nullptr : ws.get<float>((size_t)H * max_active);
  if (!ws.ok) return FOCUS_ERR_WORKSPACE_TOO_SMALL;
  const bool tc = !ctx->force_simt && sink_tc_supported(ctx, shape, max_active);
  if (!lse) {
    // no log-sum-exp from a dense pass: compute it here (one extra pass over K, no values read)
    AttnArgs a{};
    a.sh = *shape; a.scale = shape_scale(shape);
    a.Q = Q; a.q_base = q_base; a.n_q = L - q_base; a.q_rows = active_idx; a.n_rows = n_active;
    a.max_rows = max_active; a.K = K; a.V = K; a.O = nullptr; a.lse = lse_buf; a.lse_stride = max_active; a.dense = 1;
    focus_status s;
    if (tc) {
      // the tensor-core attention kernel yields the LSE as a by-product; its output rows (with K standing in for V)
      // go to scratch and are dropped
      a.O = ws.get<__nv_bfloat16>((size_t)max_active * H * shape->head_dim);
      if (!ws.ok) return FOCUS_ERR_WORKSPACE_TOO_SMALL;
      s = attn_tc_supported(ctx, a) ? launch_attn_tc_ws(ctx, a, ws, nullptr, stream) : FOCUS_ERR_UNSUPPORTED;
      if (s == FOCUS_ERR_UNSUPPORTED) { a.O = nullptr; s = launch_attn_simt(ctx, a, stream); }
    } else {
      s = launch_attn_simt(ctx, a, stream);
    }
    if (s != FOCUS_OK) return s;
    lse = lse_buf;
  }
  focus_status s;
  if (tc) s = launch_sink_colsum_tc(ctx, shape, Q, q_base, active_idx, n_active, max_active, K, lse, part, ws, stream);
  else s = launch_sink_colsum_simt(ctx, shape, Q, q_base, active_idx, n_active, max_active, K, lse, part, stream);
  if (s != FOCUS_OK) return s;
  return launch_sink_select(ctx, part, H, L, n_active, S, cand_lo, cand_hi, n_sink, sink_idx, stream);
}

extern "C" focus_status focus_select_sinks(focus_ctx* ctx, const float* scores, int32_t L, int32_t cand_lo,
                                           int32_t cand_hi, int32_t n_sink, int32_t* sink_idx, focus_stream stream) {
  FOCUS_STAGE("focus_select_sinks");
  if (!ctx || !scores || L <= 0 || n_sink < 0 || (n_sink > 0 && !sink_idx)) return FOCUS_ERR_INVALID_ARG;
  if (cand_lo < 0 || cand_hi < cand_lo || cand_hi > L) return FOCUS_ERR_INVALID_ARG;
  if (n_sink == 0) return FOCUS_OK;
  return launch_sink_topn(ctx, scores, nullptr, cand_lo, cand_hi, n_sink, sink_idx, (cudaStream_t)stream);
}

