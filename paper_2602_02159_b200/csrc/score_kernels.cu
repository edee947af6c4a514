// Block-importance scorer: mean-pooled key blocks K-bar_b and block relevance R_b (Eq. 7).
// R is linear in the queries, so R[g][b] = qbar[g] . Kbar[g][b] with qbar[g] the mean of the focus rows over
// the query heads of KV head g.  The cold path streams the prompt keys once (HBM-bound) and never
// materialises K-bar; the warm path reads a cached K-bar.
#include "focus_common.cuh"

// qbar[g][c] = mean over focus rows i and heads h of group g of Q[i][h][c]   (fp32, fixed order)
template <typename T>
__global__ void qbar_kernel(const T* __restrict__ Q, int q_base, int n_q_rows_bound, long long q_stride_row,
                            long long q_stride_head, const int32_t* __restrict__ focus_idx,
                            const int32_t* __restrict__ n_focus, int max_focus, int hpg, int d, int L,
                            float* __restrict__ qbar, int32_t* status) {
  const int g = blockIdx.x;
  const int c = threadIdx.x;
  if (c >= d) return;
  int nf = *n_focus;
  if (nf > max_focus) nf = max_focus;
  float acc = 0.f;
  int cnt = 0;
  for (int i = 0; i < nf; ++i) {
    const int pos = focus_idx[i];
    if (pos < q_base || pos >= L) {
      if (c == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
      continue;
    }
    const T* row = Q + (long long)(pos - q_base) * q_stride_row;
    for (int hh = 0; hh < hpg; ++hh) acc += load_as_float(row + (long long)(g * hpg + hh) * q_stride_head + c);
    ++cnt;
  }
  if (c == 0 && cnt == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
  qbar[g * d + c] = cnt > 0 ? acc / (float)(cnt * hpg) : 0.f;
}

// One CTA per (block b, KV head g): 256 threads, each owning one 16-byte column chunk and striding over rows.
// Writes Kbar (if non-NULL) and/or R[g][b] = qbar[g] . mean (if qbar non-NULL).
template <typename T, int D>
__device__ __forceinline__ void pool_score_block(const T* __restrict__ K, long long kv_stride_tok, long long kv_stride_head,
                                                 int M, int B, int nb, float* __restrict__ Kbar,
                                                 const float* __restrict__ qbar, float* __restrict__ R, int b, int g) {
  constexpr int EPC = 16 / sizeof(T);          // elements per 16-byte chunk
  constexpr int CPR = D / EPC;                 // chunks per row
  constexpr int RPI = 256 / CPR;               // rows per iteration
  __shared__ float red[RPI][D + 1];
  __shared__ float dotp[8];
  const int lo = b * B, hi = min(lo + B, M);
  const int chunk = threadIdx.x % CPR, rsub = threadIdx.x / CPR;
  float acc[EPC];
#pragma unroll
  for (int e = 0; e < EPC; ++e) acc[e] = 0.f;
  const T* base = K + (long long)g * kv_stride_head + chunk * EPC;
#pragma unroll 4
  for (int j = lo + rsub; j < hi; j += RPI) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(base + (long long)j * kv_stride_tok));
    if constexpr (sizeof(T) == 2) {
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(p[e]);
        acc[2 * e] += f.x;
        acc[2 * e + 1] += f.y;
      }
    } else {
      const float* p = reinterpret_cast<const float*>(&raw);
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[e] += p[e];
    }
  }
#pragma unroll
  for (int e = 0; e < EPC; ++e) red[rsub][chunk * EPC + e] = acc[e];
  __syncthreads();
  float dot = 0.f;
  if (threadIdx.x < D) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < RPI; ++r) s += red[r][threadIdx.x];
    const float mean = s / (float)(hi - lo);
    if (Kbar) Kbar[((size_t)g * nb + b) * D + threadIdx.x] = mean;
    if (qbar) dot = mean * qbar[g * D + threadIdx.x];
  }
  if (qbar) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if ((threadIdx.x & 31) == 0) dotp[threadIdx.x >> 5] = dot;
    __syncthreads();
    if (threadIdx.x == 0) {
      float s = 0.f;
      for (int w2 = 0; w2 < D / 32; ++w2) s += dotp[w2];
      R[(size_t)g * nb + b] = s;
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(256)
pool_score_kernel(const T* __restrict__ K, long long kv_stride_tok, long long kv_stride_head, int M, int B, int nb,
                  float* __restrict__ Kbar, const float* __restrict__ qbar, float* __restrict__ R) {
  pool_score_block<T, D>(K, kv_stride_tok, kv_stride_head, M, B, nb, Kbar, qbar, R, blockIdx.x, blockIdx.y);
  publish_outputs();
}

// Incremental maintenance of the pooled keys after a KV-cache refresh (Eq. 3): grid (max_rows, Hkv); CTA (r, g)
// re-pools the prompt block that holds refreshed position rows[r] for KV head g, with the arithmetic of the full
// pooling kernel (same reduction order: the result is bit-identical to pooling everything again).  Rows in the
// response region touch no pooled key.  With an ascending list the CTA of the first listed row of a block does the
// work and the others of that block leave; an unsorted list only costs repeated, identical work.
template <typename T, int D>
__global__ void __launch_bounds__(256)
pool_rows_kernel(const T* __restrict__ K, long long kv_stride_tok, long long kv_stride_head, int M, int B, int nb,
                 const int32_t* __restrict__ rows, const int32_t* __restrict__ n_rows, int max_rows,
                 float* __restrict__ Kbar, int32_t* status) {
  const int r = blockIdx.x, g = blockIdx.y;
  const int n = min(max(*n_rows, 0), max_rows);
  if (r >= n) return;
  const int pos = rows[r];
  if (pos < 0) {
    if (threadIdx.x == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
    return;
  }
  if (pos >= M) return;
  const int b = pos / B;
  if (r > 0) {
    const int prev = rows[r - 1];
    if (prev >= 0 && prev < M && prev / B == b) return;
  }
  pool_score_block<T, D>(K, kv_stride_tok, kv_stride_head, M, B, nb, Kbar, nullptr, nullptr, b, g);
  publish_outputs();
}

// Warm path: one warp per (block, group): R[g][b] = qbar[g] . Kbar[g][b].
__global__ void score_from_kbar_kernel(const float* __restrict__ Kbar, const float* __restrict__ qbar, int nb, int d,
                                       int G, float* __restrict__ R) {
  const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (wid >= nb * G) return;
  const int g = wid / nb;
  const float* kb = Kbar + (size_t)wid * d;
  float s = 0.f;
  for (int c = lane; c < d; c += 32) s += kb[c] * qbar[g * d + c];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) R[wid] = s;
}

// ALL-heads mode: R[b] = mean over groups of Rg[g][b] (groups have equal size, so this is the mean over heads).
__global__ void reduce_groups_kernel(const float* __restrict__ Rg, int G, int nb, float* __restrict__ R) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= nb) return;
  float s = 0.f;
  for (int g = 0; g < G; ++g) s += Rg[(size_t)g * nb + b];
  R[b] = s / (float)G;
}

template <typename T>
static focus_status pool_score_launch(const focus_shape* s, const void* K, float* Kbar, const float* qbar, float* R,
                                      cudaStream_t st) {
  const int nb = shape_nb(s);
  if (nb == 0) return FOCUS_OK;
  dim3 grid(nb, s->n_kv_heads);
  if (s->head_dim == 128)
    pool_score_kernel<T, 128><<<grid, 256, 0, st>>>((const T*)K, s->kv_stride_tok, s->kv_stride_head, s->M,
                                                    s->kv_block, nb, Kbar, qbar, R);
  else
    pool_score_kernel<T, 64><<<grid, 256, 0, st>>>((const T*)K, s->kv_stride_tok, s->kv_stride_head, s->M,
                                                   s->kv_block, nb, Kbar, qbar, R);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}

extern "C" focus_status focus_pool_keys(focus_ctx* ctx, const focus_shape* shape, const void* K, float* Kbar,
                                        focus_stream stream) {
  FOCUS_STAGE("focus_pool_keys");
  if (!ctx || !shape_ok_basic(shape) || !K || !Kbar || !all_aligned16(K, Kbar)) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;
  return shape->dtype == FOCUS_BF16 ? pool_score_launch<__nv_bfloat16>(shape, K, Kbar, nullptr, nullptr, stream)
                                    : pool_score_launch<float>(shape, K, Kbar, nullptr, nullptr, stream);
}

extern "C" focus_status focus_update_pooled_keys(focus_ctx* ctx, const focus_shape* shape, const void* K, float* Kbar,
                                                 const int32_t* rows, const int32_t* n_rows, int32_t max_rows,
                                                 focus_stream stream) {
  FOCUS_STAGE("focus_update_pooled_keys");
  if (!ctx || !shape_ok_basic(shape) || !K || !Kbar || !rows || !n_rows || !all_aligned16(K, Kbar)) return FOCUS_ERR_INVALID_ARG;
  if (max_rows < 0) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;
  const int nb = shape_nb(shape);
  if (max_rows == 0 || nb == 0) return FOCUS_OK;
  dim3 grid(max_rows, shape->n_kv_heads);
  const long long st = shape->kv_stride_tok, sh = shape->kv_stride_head;
  const int M = shape->M, B = shape->kv_block;
  if (shape->dtype == FOCUS_BF16) {
    if (shape->head_dim == 128)
      pool_rows_kernel<__nv_bfloat16, 128><<<grid, 256, 0, stream>>>((const __nv_bfloat16*)K, st, sh, M, B, nb, rows, n_rows, max_rows, Kbar, ctx->d_status);
    else
      pool_rows_kernel<__nv_bfloat16, 64><<<grid, 256, 0, stream>>>((const __nv_bfloat16*)K, st, sh, M, B, nb, rows, n_rows, max_rows, Kbar, ctx->d_status);
  } else {
    if (shape->head_dim == 128)
      pool_rows_kernel<float, 128><<<grid, 256, 0, stream>>>((const float*)K, st, sh, M, B, nb, rows, n_rows, max_rows, Kbar, ctx->d_status);
    else
      pool_rows_kernel<float, 64><<<grid, 256, 0, stream>>>((const float*)K, st, sh, M, B, nb, rows, n_rows, max_rows, Kbar, ctx->d_status);
  }
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}

extern "C" focus_status focus_score_blocks(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base,
                                           const int32_t* focus_idx, const int32_t* n_focus, int32_t max_focus,
                                           const void* K, const float* Kbar, int32_t head_reduce, float* R,
                                           focus_stream stream) {
  FOCUS_STAGE("focus_score_blocks");
  if (!ctx || !shape_ok_basic(shape) || !Q || !focus_idx || !n_focus || !R) return FOCUS_ERR_INVALID_ARG;
  if ((K == nullptr) == (Kbar == nullptr) || !all_aligned16(Q, K, Kbar)) return FOCUS_ERR_INVALID_ARG;
  if (max_focus <= 0 || q_base < 0 || q_base > shape->L) return FOCUS_ERR_INVALID_ARG;
  if (head_reduce != FOCUS_HEADS_PER_KV_GROUP && head_reduce != FOCUS_HEADS_ALL) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;
  const int G = shape->n_kv_heads, d = shape->head_dim, nb = shape_nb(shape), hpg = shape->n_q_heads / G;
  WsAlloc ws(ctx);
  float* qbar = ws.get<float>((size_t)G * d);
  float* Rg = head_reduce == FOCUS_HEADS_ALL ? ws.get<float>((size_t)G * nb) : R;
  if (!ws.ok) return FOCUS_ERR_WORKSPACE_TOO_SMALL;
  if (shape->dtype == FOCUS_BF16)
    qbar_kernel<__nv_bfloat16><<<G, 128, 0, stream>>>((const __nv_bfloat16*)Q, q_base, 0, shape->q_stride_row,
                                                      shape->q_stride_head, focus_idx, n_focus, max_focus, hpg, d,
                                                      shape->L, qbar, ctx->d_status);
  else
    qbar_kernel<float><<<G, 128, 0, stream>>>((const float*)Q, q_base, 0, shape->q_stride_row, shape->q_stride_head,
                                              focus_idx, n_focus, max_focus, hpg, d, shape->L, qbar, ctx->d_status);
  FOCUS_CHECK_LAUNCH();
  if (nb == 0) return FOCUS_OK;
  if (K) {
    focus_status st = shape->dtype == FOCUS_BF16 ? pool_score_launch<__nv_bfloat16>(shape, K, nullptr, qbar, Rg, stream)
                                                 : pool_score_launch<float>(shape, K, nullptr, qbar, Rg, stream);
    if (st != FOCUS_OK) return st;
  } else {
    const int warps = nb * G;
    score_from_kbar_kernel<<<(warps * 32 + 255) / 256, 256, 0, stream>>>(Kbar, qbar, nb, d, G, Rg);
    FOCUS_CHECK_LAUNCH();
  }
  if (head_reduce == FOCUS_HEADS_ALL) {
    reduce_groups_kernel<<<(nb + 255) / 256, 256, 0, stream>>>(Rg, G, nb, R);
    FOCUS_CHECK_LAUNCH();
  }
  return FOCUS_OK;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of focus_score_blocks.
//
// Written for callers that must never allocate device memory: code running inside someone else's memory
// budget (an inference server whose pool already owns the whole GPU), code on a path where cudaMalloc's
// implicit device synchronisation is unacceptable, or a plug-in that is handed a stream and nothing else.
// Such callers cannot create a focus_ctx either (focus_create allocates the workspace), so this entry point
// takes no context.  Its scratch -- the mean focus query of every KV head and, in all-heads mode, the
// per-group scores before they are averaged -- lives in the fixed array below, which every GPU that loads the
// library holds until the process exits.
// ------------------------------------------------------------------------------------------------
constexpr int STATIC_QBAR_FLOATS = 64 * 128;        // n_kv_heads * head_dim        <= 8192
constexpr int STATIC_RG_FLOATS = 64 * 1024;         // n_kv_heads * nb (ALL mode)   <= 65536
constexpr int STATIC_SCRATCH_FLOATS = STATIC_QBAR_FLOATS + STATIC_RG_FLOATS + 64;   // + status word; 288.25 KiB

static __device__ __align__(256) float g_static_scratch[STATIC_SCRATCH_FLOATS];

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel may use: the device
// address is looked up once per device (with that device current) and cached here.  The cache is written without a
// lock: two host threads racing on a device's first call both store the same address, so whichever store lands
// last changes nothing.  That first lookup also makes the runtime load this module onto the device (which is where
// the array gets its memory), one more reason to make the first call outside any stream capture.
constexpr int STATIC_MAX_DEVICES = 64;
static float* g_static_scratch_dev[STATIC_MAX_DEVICES] = {nullptr};

static focus_status static_scratch_ptr(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return FOCUS_ERR_CUDA;
  if (!g_static_scratch_dev[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return FOCUS_ERR_CUDA;
    g_static_scratch_dev[dev] = static_cast<float*>(p);
  }
  *out = g_static_scratch_dev[dev];
  return FOCUS_OK;
}

extern "C" focus_status focus_score_blocks_static(const focus_shape* shape, const void* Q, int32_t q_base,
                                                  const int32_t* focus_idx, const int32_t* n_focus,
                                                  int32_t max_focus, const void* K, const float* Kbar,
                                                  int32_t head_reduce, float* R, int32_t* device_status,
                                                  focus_stream stream) {
  if (!shape_ok_basic(shape) || !Q || !focus_idx || !n_focus || !R) return FOCUS_ERR_INVALID_ARG;
  if ((K == nullptr) == (Kbar == nullptr) || !all_aligned16(Q, K, Kbar)) return FOCUS_ERR_INVALID_ARG;
  if (max_focus <= 0 || q_base < 0 || q_base > shape->L) return FOCUS_ERR_INVALID_ARG;
  if (head_reduce != FOCUS_HEADS_PER_KV_GROUP && head_reduce != FOCUS_HEADS_ALL) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;
  const int G = shape->n_kv_heads, d = shape->head_dim, nb = shape_nb(shape), hpg = shape->n_q_heads / G;
  // the fixed scratch bounds the problem size: refuse anything that would not fit
  if ((long long)G * d > STATIC_QBAR_FLOATS) return FOCUS_ERR_WORKSPACE_TOO_SMALL;
  if (head_reduce == FOCUS_HEADS_ALL && (long long)G * nb > STATIC_RG_FLOATS) return FOCUS_ERR_WORKSPACE_TOO_SMALL;
  float* scratch = nullptr;
  focus_status st = static_scratch_ptr(&scratch);
  if (st != FOCUS_OK) return st;
  float* qbar = scratch;                                         // fully rewritten by every call
  float* Rg = head_reduce == FOCUS_HEADS_ALL ? scratch + STATIC_QBAR_FLOATS : R;
  int32_t* status = device_status ? device_status
                                  : reinterpret_cast<int32_t*>(scratch + STATIC_QBAR_FLOATS + STATIC_RG_FLOATS);
  if (shape->dtype == FOCUS_BF16)
    qbar_kernel<__nv_bfloat16><<<G, 128, 0, stream>>>((const __nv_bfloat16*)Q, q_base, 0, shape->q_stride_row,
                                                      shape->q_stride_head, focus_idx, n_focus, max_focus, hpg, d,
                                                      shape->L, qbar, status);
  else
    qbar_kernel<float><<<G, 128, 0, stream>>>((const float*)Q, q_base, 0, shape->q_stride_row, shape->q_stride_head,
                                              focus_idx, n_focus, max_focus, hpg, d, shape->L, qbar, status);
  FOCUS_CHECK_LAUNCH();
  if (nb == 0) return FOCUS_OK;
  if (K) {
    st = shape->dtype == FOCUS_BF16 ? pool_score_launch<__nv_bfloat16>(shape, K, nullptr, qbar, Rg, stream)
                                    : pool_score_launch<float>(shape, K, nullptr, qbar, Rg, stream);
    if (st != FOCUS_OK) return st;
  } else {
    const int warps = nb * G;
    score_from_kbar_kernel<<<(warps * 32 + 255) / 256, 256, 0, stream>>>(Kbar, qbar, nb, d, G, Rg);
    FOCUS_CHECK_LAUNCH();
  }
  if (head_reduce == FOCUS_HEADS_ALL) {
    reduce_groups_kernel<<<(nb + 255) / 256, 256, 0, stream>>>(Rg, G, nb, R);
    FOCUS_CHECK_LAUNCH();
  }
  return FOCUS_OK;
}
