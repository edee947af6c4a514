// The per-step pieces that close the decoding loop around the attention path:
//   focus_confidence  -- Eq. 2: predicted token and confidence c = max_v softmax(logits)_v of the active rows
//                        (an HBM-bound streaming reduction over the vocabulary; its output is the conf_prev of the
//                        next step's focus_select_queries, and with k = n, w = 0 the same call picks the tokens
//                        to unmask);
//   focus_update_kv   -- Eq. 3; Algorithm 1, the cache-update step of the non-block-entry branch: the refreshed
//                        rows replace the cached K and V rows;
//   focus_commit_step -- Algorithm 1, the state update at the end of a step, with the unmasking rule stated after
//                        Eq. 2: the new confidences of the evaluated rows enter the confidence vector, the n most
//                        confident still-masked evaluated positions of the decoding block receive their predicted
//                        tokens and leave the masked set.
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
  publish_outputs();
}

constexpr int CS_THREADS = 1024;
constexpr int CS_MAX_ROWS = 4096;

// One CTA.  Row r of (conf_new, token_new) belongs to position rows[r] (or pos_base + r).  Candidates for unmasking:
// evaluated positions that are still masked and lie in [blk_lo, blk_hi); the n_unmask with the highest new confidence
// win (ties: lower row, i.e. lower position for an ascending list; NaN last).  Every read of masked[] precedes every
// write (one CTA, barriers in between).
__global__ void __launch_bounds__(CS_THREADS)
commit_step_kernel(const float* __restrict__ conf_new, const int32_t* __restrict__ token_new, int pos_base,
                   const int32_t* __restrict__ rows, const int32_t* __restrict__ n_rows, int max_rows, int L, int blk_lo,
                   int blk_hi, int n_unmask, float* __restrict__ conf, uint8_t* __restrict__ masked,
                   int32_t* __restrict__ x, int32_t* __restrict__ unmasked_idx, int32_t* __restrict__ n_unmasked,
                   int32_t* status) {
  __shared__ uint32_t ckey[CS_MAX_ROWS];     // compacted candidates: order-preserving confidence key,
  __shared__ int crow[CS_MAX_ROWS];          // the row they came from (ascending)
  __shared__ uint8_t sel[CS_MAX_ROWS];
  __shared__ int scan_s[33];
  __shared__ int hist[258];
  const int tid = threadIdx.x;
  const int n = rows ? min(max(*n_rows, 0), max_rows) : max_rows;
  int base = 0;
  for (int r0 = 0; r0 < n; r0 += CS_THREADS) {
    const int r = r0 + tid;
    int is_cand = 0, pos = -1;
    float c = 0.f;
    if (r < n) {
      pos = rows ? rows[r] : pos_base + r;
      if (pos < 0 || pos >= L) {
        set_status(status, FOCUS_ERR_INVALID_ARG);
        pos = -1;
      } else {
        c = conf_new[r];
        is_cand = (masked[pos] != 0 && pos >= blk_lo && pos < blk_hi) ? 1 : 0;
      }
    }
    int tot;
    const int pre = block_excl_scan(is_cand, scan_s, tot);
    if (is_cand) { ckey[base + pre] = float_key(c); crow[base + pre] = r; }
    base += tot;
  }
  __syncthreads();
  const int n_cand = base;
  const int n_take = min(max(n_unmask, 0), n_cand);
  block_topc_mark(ckey, n_cand, n_take, sel, hist, scan_s);
  // the new confidences enter the vector (every evaluated position, masked or not)
  for (int r = tid; r < n; r += CS_THREADS) {
    const int pos = rows ? rows[r] : pos_base + r;
    if (pos >= 0 && pos < L) conf[pos] = conf_new[r];
  }
  // winners: token written, mask cleared, position reported (ascending)
  int out_base = 0;
  for (int j0 = 0; j0 < n_cand; j0 += CS_THREADS) {
    const int j = j0 + tid;
    const int f = (j < n_cand && sel[j]) ? 1 : 0;
    int tot;
    const int pre = block_excl_scan(f, scan_s, tot);
    if (f) {
      const int r = crow[j];
      const int pos = rows ? rows[r] : pos_base + r;
      x[pos] = token_new[r];
      masked[pos] = 0;
      if (unmasked_idx) unmasked_idx[out_base + pre] = pos;
    }
    out_base += tot;
  }
  if (unmasked_idx)
    for (int i = out_base + tid; i < n_unmask; i += CS_THREADS) unmasked_idx[i] = -1;
  if (tid == 0 && n_unmasked) *n_unmasked = out_base;
}

}  // namespace

extern "C" focus_status focus_confidence(focus_ctx* ctx, const void* logits, int32_t dtype, int64_t row_stride,
                                         int32_t vocab, int32_t pos_base, int32_t n_pos, const int32_t* rows,
                                         const int32_t* n_rows, int32_t max_rows, float* conf, int32_t* token,
                                         focus_stream stream) {
  FOCUS_STAGE("focus_confidence");
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
  FOCUS_STAGE("focus_update_kv");
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

extern "C" focus_status focus_commit_step(focus_ctx* ctx, const float* conf_new, const int32_t* token_new,
                                          int32_t pos_base, const int32_t* rows, const int32_t* n_rows,
                                          int32_t max_rows, int32_t L, int32_t blk_lo, int32_t blk_hi,
                                          int32_t n_unmask, float* conf, uint8_t* masked, int32_t* x,
                                          int32_t* unmasked_idx, int32_t* n_unmasked, focus_stream stream) {
  FOCUS_STAGE("focus_commit_step");
  if (!ctx || !conf_new || !token_new || !conf || !masked || !x) return FOCUS_ERR_INVALID_ARG;
  if ((rows == nullptr) != (n_rows == nullptr)) return FOCUS_ERR_INVALID_ARG;
  if (L <= 0 || pos_base < 0 || max_rows < 0 || max_rows > CS_MAX_ROWS || n_unmask < 0 || n_unmask > CS_MAX_ROWS)
    return FOCUS_ERR_INVALID_ARG;
  if (blk_lo < 0 || blk_hi < blk_lo || blk_hi > L) return FOCUS_ERR_INVALID_ARG;
  if (!rows && pos_base + max_rows > L) return FOCUS_ERR_INVALID_ARG;
  if (n_unmask > 0 && !unmasked_idx) return FOCUS_ERR_INVALID_ARG;
  commit_step_kernel<<<1, CS_THREADS, 0, stream>>>(conf_new, token_new, pos_base, rows, n_rows, max_rows, L, blk_lo,
                                                  blk_hi, n_unmask, conf, masked, x, unmasked_idx, n_unmasked,
                                                  ctx->d_status);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}
