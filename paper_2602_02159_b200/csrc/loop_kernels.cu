// The two per-step pieces that close the decoding loop around the attention path:
//   focus_confidence  -- Eq. 2: predicted token and confidence c = max_v softmax(logits)_v of the active rows
//                        (an HBM-bound streaming reduction over the vocabulary; its output is the conf_prev of the
//                        next step's focus_select_queries, and with k = n, w = 0 the same call picks the tokens
//                        to unmask);
//   focus_update_kv   -- Eq. 3; Algorithm 1, the cache-update step of the non-block-entry branch: the refreshed
//                        rows replace the cached K and V rows.
#include "focus_common.cuh"

namespace {

struct Msi {      // running maximum, sum of exp(x - m), index of the maximum (lowest index on ties)
  float m, s;
  int i;
};

__device__ __forceinline__ Msi msi_merge(const Msi& a, const Msi& b) {
  Msi r;
  if (a.m == -INFINITY && b.m == -INFINITY) { r.m = -INFINITY; r.s = 0.f; r.i = min(a.i, b.i); return r; }
  r.m = fmaxf(a.m, b.m);
  r.s = a.s * __expf(a.m - r.m) + b.s * __expf(b.m - r.m);
  r.i = a.m > b.m ? a.i : (b.m > a.m ? b.i : min(a.i, b.i));
  return r;
}

constexpr int CF_THREADS = 256;

// grid (chunks, max_rows): CTA (c, r) reduces elements [c*per, (c+1)*per) of row r to one (m, s, i) triple.
template <typename T>
__global__ void __launch_bounds__(CF_THREADS)
confidence_partial_kernel(const T* __restrict__ logits, long long row_stride, int vocab, int pos_base, int n_pos,
                          const int32_t* __restrict__ rows, const int32_t* __restrict__ n_rows, int max_rows,
                          int per, Msi* __restrict__ part, int32_t* status) {
  constexpr int EPC = 16 / sizeof(T);
  __shared__ Msi red[CF_THREADS / 32];
  const int r = blockIdx.y, c = blockIdx.x;
  const int n = rows ? min(max(*n_rows, 0), max_rows) : max_rows;
  if (r >= n) return;
  const int pos = rows ? rows[r] : pos_base + r;
  Msi acc; acc.m = -INFINITY; acc.s = 0.f; acc.i = 0x7fffffff;
  if (pos < pos_base || pos >= pos_base + n_pos) {
    if (threadIdx.x == 0) { set_status(status, FOCUS_ERR_INVALID_ARG); part[(size_t)r * gridDim.x + c] = acc; }
    return;
  }
  const T* row = logits + (long long)(pos - pos_base) * row_stride;
  const int lo = c * per, hi = min(lo + per, vocab);
  for (int v0 = lo + threadIdx.x * EPC; v0 < hi; v0 += CF_THREADS * EPC) {
    float x[EPC];
    if (v0 + EPC <= hi) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(row + v0));
      if constexpr (sizeof(T) == 2) {
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int e = 0; e < 4; ++e) { const float2 f = __bfloat1622float2(p2[e]); x[2 * e] = f.x; x[2 * e + 1] = f.y; }
      } else {
        const float* pf = reinterpret_cast<const float*>(&raw);
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = pf[e];
      }
    } else {
#pragma unroll
      for (int e = 0; e < EPC; ++e) x[e] = v0 + e < hi ? load_as_float(row + v0 + e) : -INFINITY;
    }
    // local maximum of the chunk first, then one rescale of the running sum
    float cm = -INFINITY;
    int ci = 0;
#pragma unroll
    for (int e = 0; e < EPC; ++e) {
      const float xe = x[e] != x[e] ? -INFINITY : x[e];          // NaN counts as -inf
      x[e] = xe;
      if (xe > cm) { cm = xe; ci = e; }
    }
    if (cm == -INFINITY) continue;
    if (cm > acc.m) { acc.s *= __expf(acc.m - cm); acc.m = cm; acc.i = v0 + ci; }
#pragma unroll
    for (int e = 0; e < EPC; ++e) acc.s += __expf(x[e] - acc.m);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Msi b;
    b.m = __shfl_xor_sync(0xffffffffu, acc.m, o);
    b.s = __shfl_xor_sync(0xffffffffu, acc.s, o);
    b.i = __shfl_xor_sync(0xffffffffu, acc.i, o);
    acc = msi_merge(acc, b);
  }
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    Msi t = red[0];
    for (int w2 = 1; w2 < CF_THREADS / 32; ++w2) t = msi_merge(t, red[w2]);
    part[(size_t)r * gridDim.x + c] = t;
  }
}

// one thread per row merges the row's chunk triples in chunk order
__global__ void confidence_final_kernel(const Msi* __restrict__ part, int chunks, const int32_t* __restrict__ rows,
                                        const int32_t* __restrict__ n_rows, int max_rows, float* __restrict__ conf,
                                        int32_t* __restrict__ token) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= max_rows) return;
  const int n = rows ? min(max(*n_rows, 0), max_rows) : max_rows;
  if (r >= n) { conf[r] = 0.f; token[r] = -1; return; }
  Msi t = part[(size_t)r * chunks];
  for (int c = 1; c < chunks; ++c) t = msi_merge(t, part[(size_t)r * chunks + c]);
  conf[r] = t.s > 0.f ? 1.f / t.s : 0.f;
  token[r] = t.s > 0.f ? t.i : -1;
}

// grid (max_rows, Hkv): one 16-byte chunk of K and of V per thread
template <typename T>
__global__ void update_kv_kernel(T* __restrict__ Kc, T* __restrict__ Vc, const T* __restrict__ Kn,
                                 const T* __restrict__ Vn, long long kv_stride_tok, long long kv_stride_head, int L,
                                 int Hkv, int d, const int32_t* __restrict__ rows, const int32_t* __restrict__ n_rows,
                                 int max_rows, int32_t* status) {
  constexpr int EPC = 16 / sizeof(T);
  const int r = blockIdx.x, g = blockIdx.y;
  const int n = min(max(*n_rows, 0), max_rows);
  if (r >= n) return;
  const int pos = rows[r];
  if (pos < 0 || pos >= L) {
    if (threadIdx.x == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
    return;
  }
  const int c = threadIdx.x;
  if (c * EPC >= d) return;
  const size_t src = ((size_t)r * Hkv + g) * d + c * EPC;
  const size_t dst = (size_t)g * kv_stride_head + (size_t)pos * kv_stride_tok + c * EPC;
  *reinterpret_cast<uint4*>(Kc + dst) = __ldg(reinterpret_cast<const uint4*>(Kn + src));
  *reinterpret_cast<uint4*>(Vc + dst) = __ldg(reinterpret_cast<const uint4*>(Vn + src));
}

}  // namespace

extern "C" focus_status focus_confidence(focus_ctx* ctx, const void* logits, int32_t dtype, int64_t row_stride,
                                         int32_t vocab, int32_t pos_base, int32_t n_pos, const int32_t* rows,
                                         const int32_t* n_rows, int32_t max_rows, float* conf, int32_t* token,
                                         focus_stream stream) {
  if (!ctx || !logits || !conf || !token || !aligned16(logits)) return FOCUS_ERR_INVALID_ARG;
  if (dtype != FOCUS_F32 && dtype != FOCUS_BF16) return FOCUS_ERR_INVALID_ARG;
  if (vocab <= 0 || row_stride < vocab || pos_base < 0 || n_pos < 0 || max_rows < 0) return FOCUS_ERR_INVALID_ARG;
  if ((rows == nullptr) != (n_rows == nullptr)) return FOCUS_ERR_INVALID_ARG;
  if (!rows && max_rows > n_pos) return FOCUS_ERR_INVALID_ARG;
  const int epc = dtype == FOCUS_BF16 ? 8 : 4;
  if (row_stride % epc) return FOCUS_ERR_INVALID_ARG;            // rows must keep 16-byte alignment
  if (max_rows == 0) return FOCUS_OK;
  // enough chunks per row to occupy the GPU about twice over, each a multiple of one CTA sweep
  int chunks = (2 * ctx->sm_count + max_rows - 1) / max_rows;
  const int sweep = CF_THREADS * epc;
  const int max_chunks = (vocab + sweep - 1) / sweep;
  if (chunks > max_chunks) chunks = max_chunks;
  if (chunks < 1) chunks = 1;
  int per = ((vocab + chunks - 1) / chunks + sweep - 1) / sweep * sweep;
  chunks = (vocab + per - 1) / per;
  WsAlloc ws(ctx);
  Msi* part = ws.get<Msi>((size_t)max_rows * chunks);
  if (!ws.ok) return FOCUS_ERR_WORKSPACE_TOO_SMALL;
  dim3 grid(chunks, max_rows);
  if (dtype == FOCUS_BF16)
    confidence_partial_kernel<__nv_bfloat16><<<grid, CF_THREADS, 0, stream>>>(
        (const __nv_bfloat16*)logits, row_stride, vocab, pos_base, n_pos, rows, n_rows, max_rows, per, part, ctx->d_status);
  else
    confidence_partial_kernel<float><<<grid, CF_THREADS, 0, stream>>>((const float*)logits, row_stride, vocab, pos_base,
                                                                      n_pos, rows, n_rows, max_rows, per, part,
                                                                      ctx->d_status);
  FOCUS_CHECK_LAUNCH();
  confidence_final_kernel<<<(max_rows + 127) / 128, 128, 0, stream>>>(part, chunks, rows, n_rows, max_rows, conf, token);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}

extern "C" focus_status focus_update_kv(focus_ctx* ctx, const focus_shape* shape, void* K_cache, void* V_cache,
                                        const void* K_new, const void* V_new, const int32_t* rows,
                                        const int32_t* n_rows, int32_t max_rows, focus_stream stream) {
  if (!ctx || !shape_ok_basic(shape) || !K_cache || !V_cache || !K_new || !V_new || !rows || !n_rows)
    return FOCUS_ERR_INVALID_ARG;
  if (!all_aligned16(K_cache, V_cache, K_new, V_new)) return FOCUS_ERR_INVALID_ARG;
  if (max_rows < 0) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;
  if (max_rows == 0) return FOCUS_OK;
  dim3 grid(max_rows, shape->n_kv_heads);
  if (shape->dtype == FOCUS_BF16)
    update_kv_kernel<__nv_bfloat16><<<grid, 32, 0, stream>>>((__nv_bfloat16*)K_cache, (__nv_bfloat16*)V_cache,
                                                            (const __nv_bfloat16*)K_new, (const __nv_bfloat16*)V_new,
                                                            shape->kv_stride_tok, shape->kv_stride_head, shape->L,
                                                            shape->n_kv_heads, shape->head_dim, rows, n_rows, max_rows,
                                                            ctx->d_status);
  else
    update_kv_kernel<float><<<grid, 32, 0, stream>>>((float*)K_cache, (float*)V_cache, (const float*)K_new,
                                                    (const float*)V_new, shape->kv_stride_tok, shape->kv_stride_head,
                                                    shape->L, shape->n_kv_heads, shape->head_dim, rows, n_rows, max_rows,
                                                    ctx->d_status);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}
