// Generic SIMT attention (Eq. 9 and FullAttn of Algorithm 1) and the SIMT sink column-sum (Eq. 6).
// Any dtype (f32, bf16), head_dim 64/128, any block size: this is the fp32 path of the library and the
// fallback for shapes the tensor-core kernels do not take.  One warp per (query row, head); the lanes of a
// warp hold 32 different keys during the logit phase and 32 slices of the output during the value phase.
#include "focus_common.cuh"

template <typename T, int D>
__device__ __forceinline__ float dot_row(const float* __restrict__ q, const T* __restrict__ kr) {
  constexpr int EPC = 16 / sizeof(T);
  float s = 0.f;
#pragma unroll 4
  for (int c = 0; c < D / EPC; ++c) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(kr) + c);
    if constexpr (sizeof(T) == 2) {
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(p[e]);
        s = fmaf(q[c * 8 + 2 * e], f.x, s);
        s = fmaf(q[c * 8 + 2 * e + 1], f.y, s);
      }
    } else {
      const float* p = reinterpret_cast<const float*>(&raw);
#pragma unroll
      for (int e = 0; e < 4; ++e) s = fmaf(q[c * 4 + e], p[e], s);
    }
  }
  return s;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

struct SimtParams {
  const void* Q; const void* K; const void* V; void* O; float* lse;
  const int32_t* q_rows; const int32_t* n_rows;
  const int32_t* block_idx; const int32_t* block_cnt; const int32_t* sink_idx; const uint8_t* sink_keep;
  long long q_stride_row, q_stride_head, kv_stride_tok, kv_stride_head;
  int q_base, n_q, rows_bound, L, M, H, hpg, B, nb, dense, group_stride, max_blocks, n_sink, lse_stride;
  float scale;
  int32_t* status;
};

template <typename T, int D>
__global__ void __launch_bounds__(128) attn_simt_kernel(const SimtParams p) {
  constexpr int EPL = D / 32;
  __shared__ float qs[4][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pair = blockIdx.x * 4 + warp;
  const int r = pair / p.H, h = pair % p.H;
  const int nrows = p.q_rows ? min(*p.n_rows, p.rows_bound) : p.n_q;
  if (r >= nrows) return;
  const int pos = p.q_rows ? p.q_rows[r] : p.q_base + r;
  if (pos < p.q_base || pos >= p.q_base + p.n_q) {
    if (lane == 0) set_status(p.status, FOCUS_ERR_INVALID_ARG);
    return;
  }
  const int g = h / p.hpg;
  const T* qrow = (const T*)p.Q + (long long)(pos - p.q_base) * p.q_stride_row + (long long)h * p.q_stride_head;
  for (int c = lane; c < D; c += 32) qs[warp][c] = load_as_float(qrow + c);
  __syncwarp();
  const T* Kg = (const T*)p.K + (long long)g * p.kv_stride_head;
  const T* Vg = (const T*)p.V + (long long)g * p.kv_stride_head;
  const bool want_o = p.O != nullptr;
  float m = -INFINITY, l = 0.f, o[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) o[e] = 0.f;

  auto step = [&](int key) {
    float s = -INFINITY;
    if (key >= 0) s = dot_row<T, D>(qs[warp], Kg + (long long)key * p.kv_stride_tok) * p.scale;
    const float mx = warp_max(s);
    if (mx == -INFINITY) return;
    const float m_new = fmaxf(m, mx);
    const float corr = expf(m - m_new);
    const float pj = key >= 0 ? expf(s - m_new) : 0.f;
    l = l * corr + warp_sum(pj);
    m = m_new;
    if (want_o) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[e] *= corr;
      for (int jj = 0; jj < 32; ++jj) {
        const float pk = __shfl_sync(0xffffffffu, pj, jj);
        const int kk = __shfl_sync(0xffffffffu, key, jj);
        if (kk >= 0) {
          const T* vr = Vg + (long long)kk * p.kv_stride_tok + lane * EPL;
#pragma unroll
          for (int e = 0; e < EPL; ++e) o[e] = fmaf(pk, load_as_float(vr + e), o[e]);
        }
      }
    }
  };
  auto span = [&](int lo, int hi) {
    for (int j0 = lo; j0 < hi; j0 += 32) step(j0 + lane < hi ? j0 + lane : -1);
  };

  if (p.dense) {
    span(0, p.L);
  } else {
    const int row = g * p.group_stride;
    const int cnt = min(p.block_cnt[row], p.max_blocks);
    for (int bi = 0; bi < cnt; ++bi) {
      const int b = p.block_idx[(size_t)row * p.max_blocks + bi];
      if (b < 0 || b >= p.nb) {
        if (lane == 0) set_status(p.status, FOCUS_ERR_INVALID_ARG);
        continue;
      }
      span(b * p.B, min((b + 1) * p.B, p.M));
    }
    for (int s0 = 0; s0 < p.n_sink; s0 += 32) {
      const int s = s0 + lane;
      int key = -1;
      if (s < p.n_sink && p.sink_keep[(size_t)row * p.n_sink + s]) {
        key = p.sink_idx[s];
        if (key < 0 || key >= p.L) {
          set_status(p.status, FOCUS_ERR_INVALID_ARG);
          key = -1;
        } else if (key >= p.M) {
          key = -1;                          // response tokens are attended below: count each key once
        }
      }
      step(key);
    }
    span(p.M, p.L);
  }
  if (want_o) {
    const float inv = l > 0.f ? 1.f / l : 0.f;
    if constexpr (sizeof(T) == 2) {
      __nv_bfloat16* orow = (__nv_bfloat16*)p.O + ((size_t)r * p.H + h) * D + lane * EPL;
#pragma unroll
      for (int e = 0; e < EPL; ++e) orow[e] = __float2bfloat16_rn(o[e] * inv);
    } else {
      float* orow = (float*)p.O + ((size_t)r * p.H + h) * D + lane * EPL;
#pragma unroll
      for (int e = 0; e < EPL; ++e) orow[e] = o[e] * inv;
    }
  }
  if (p.lse && lane == 0) p.lse[(size_t)h * p.lse_stride + r] = m + logf(l);
}

focus_status launch_attn_simt(focus_ctx* ctx, const AttnArgs& a, cudaStream_t st) {
  SimtParams p;
  p.Q = a.Q; p.K = a.K; p.V = a.V; p.O = a.O; p.lse = a.lse;
  p.q_rows = a.q_rows; p.n_rows = a.n_rows;
  p.block_idx = a.block_idx; p.block_cnt = a.block_cnt; p.sink_idx = a.sink_idx; p.sink_keep = a.sink_keep;
  p.q_stride_row = a.sh.q_stride_row; p.q_stride_head = a.sh.q_stride_head;
  p.kv_stride_tok = a.sh.kv_stride_tok; p.kv_stride_head = a.sh.kv_stride_head;
  p.q_base = a.q_base; p.n_q = a.n_q; p.rows_bound = a.max_rows; p.L = a.sh.L; p.M = a.sh.M; p.H = a.sh.n_q_heads;
  p.hpg = a.sh.n_q_heads / a.sh.n_kv_heads; p.B = a.sh.kv_block; p.nb = shape_nb(&a.sh); p.dense = a.dense;
  p.group_stride = a.group_stride; p.max_blocks = a.max_blocks; p.n_sink = a.n_sink; p.lse_stride = a.lse_stride;
  p.scale = a.scale; p.status = ctx->d_status;
  const long long pairs = (long long)a.max_rows * a.sh.n_q_heads;
  if (pairs == 0) return FOCUS_OK;
  const unsigned grid = (unsigned)((pairs + 3) / 4);
  const bool bf = a.sh.dtype == FOCUS_BF16;
  if (a.sh.head_dim == 128) {
    if (bf) attn_simt_kernel<__nv_bfloat16, 128><<<grid, 128, 0, st>>>(p);
    else attn_simt_kernel<float, 128><<<grid, 128, 0, st>>>(p);
  } else {
    if (bf) attn_simt_kernel<__nv_bfloat16, 64><<<grid, 128, 0, st>>>(p);
    else attn_simt_kernel<float, 64><<<grid, 128, 0, st>>>(p);
  }
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}

// ------------------------------------------------------------------------------------------------
// SIMT sink column-sum: part[h][j] = sum_i exp(scale * q_i^h . k_j - lse[h][i]) over the active rows.
// One thread per key (its row lives in registers), query rows staged through shared memory 32 at a time.
// ------------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(128)
sink_colsum_simt_kernel(const T* __restrict__ Q, int q_base, int q_rows_avail, long long q_stride_row,
                        long long q_stride_head, const int32_t* __restrict__ active_idx,
                        const int32_t* __restrict__ n_active, int max_active, const T* __restrict__ K,
                        long long kv_stride_tok, long long kv_stride_head, int hpg, int L, float scale,
                        const float* __restrict__ lse, int lse_stride, float* __restrict__ part, int32_t* status) {
  constexpr int RC = 32;
  __shared__ float qs[RC][D];
  __shared__ float ls[RC];
  const int h = blockIdx.y, g = h / hpg;
  const int j = blockIdx.x * 128 + threadIdx.x;
  const int n = min(*n_active, max_active);
  float kreg[D];
  if (j < L) {
    const T* kr = K + (long long)g * kv_stride_head + (long long)j * kv_stride_tok;
#pragma unroll
    for (int c = 0; c < D; ++c) kreg[c] = load_as_float(kr + c);
  }
  float acc = 0.f;
  for (int i0 = 0; i0 < n; i0 += RC) {
    const int nr = min(RC, n - i0);
    __syncthreads();
    for (int t = threadIdx.x; t < nr * D; t += 128) {
      const int i = t / D, c = t % D;
      const int pos = active_idx[i0 + i];
      float v = 0.f;
      if (pos >= q_base && pos < L)
        v = load_as_float(Q + (long long)(pos - q_base) * q_stride_row + (long long)h * q_stride_head + c);
      else if (c == 0)
        set_status(status, FOCUS_ERR_INVALID_ARG);
      qs[i][c] = v;
    }
    if (threadIdx.x < nr) ls[threadIdx.x] = lse[(size_t)h * lse_stride + i0 + threadIdx.x];
    __syncthreads();
    if (j < L) {
      for (int i = 0; i < nr; ++i) {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < D; ++c) s = fmaf(qs[i][c], kreg[c], s);
        acc += expf(s * scale - ls[i]);
      }
    }
  }
  if (j < L) part[(size_t)h * L + j] = acc;
}

focus_status launch_sink_colsum_simt(focus_ctx* ctx, const focus_shape* s, const void* Q, int q_base,
                                     const int32_t* active_idx, const int32_t* n_active, int max_active,
                                     const void* K, const float* lse, float* part, cudaStream_t st) {
  const int H = s->n_q_heads, hpg = H / s->n_kv_heads;
  dim3 grid((s->L + 127) / 128, H);
  const float scale = shape_scale(s);
#define LAUNCH_CS(T, D)                                                                                           \
  sink_colsum_simt_kernel<T, D><<<grid, 128, 0, st>>>((const T*)Q, q_base, 0, s->q_stride_row, s->q_stride_head, \
                                                      active_idx, n_active, max_active, (const T*)K,             \
                                                      s->kv_stride_tok, s->kv_stride_head, hpg, s->L, scale, lse, \
                                                      max_active, part, ctx->d_status)
  const bool bf = s->dtype == FOCUS_BF16;
  if (s->head_dim == 128) {
    if (bf) LAUNCH_CS(__nv_bfloat16, 128); else LAUNCH_CS(float, 128);
  } else {
    if (bf) LAUNCH_CS(__nv_bfloat16, 64); else LAUNCH_CS(float, 64);
  }
#undef LAUNCH_CS
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}
