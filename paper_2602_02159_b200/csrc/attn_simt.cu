// Generic SIMT attention (Eq. 9 and FullAttn of Algorithm 1) and the SIMT sink column-sum (Eq. 6).
// Any dtype (f32, bf16), head_dim 64/128, any block size: this is the fp32 path of the library and the
// fallback for shapes the tensor-core kernels do not take.  One CTA of eight or sixteen warps per (eight query rows, head); the
// lanes of a warp hold 32 different keys during the logit phase and 32 slices of the output during the value phase.
#include "focus_common.cuh"

// EPL consecutive elements of a V row as floats, one vector load
template <typename T, int EPL>
__device__ __forceinline__ void load_slice(const T* __restrict__ p, float (&out)[EPL]) {
  if constexpr (sizeof(T) == 4) {
    if constexpr (EPL == 4) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(p));
      out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    } else {
      const float2 v = __ldg(reinterpret_cast<const float2*>(p));
      out[0] = v.x; out[1] = v.y;
    }
  } else {
    if constexpr (EPL == 4) {
      const uint2 raw = __ldg(reinterpret_cast<const uint2*>(p));
      const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
      const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
      out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
    } else {
      const uint32_t raw = __ldg(reinterpret_cast<const uint32_t*>(p));
      const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw));
      out[0] = a.x; out[1] = a.y;
    }
  }
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

// warps per CTA: sixteen for head_dim 64, eight for 128 (the warps' partial outputs must fit in 48 KB)
__host__ __device__ constexpr int simt_warps(int d) { return d == 64 ? 16 : 8; }
// loads in flight per lane in the logit / value phase (deeper unrolling measured no faster: the kernel waits on L2
// latency with few warps per SM, not on issue slots)
constexpr int UNROLL_DOT = 2, UNROLL_V = 4;

// One CTA per (group of R query rows, head): the rows of a group share every K and V row that is loaded (without
// that sharing the kernel is bound by L2 bandwidth: every row would stream the head's whole K and V).  The warps
// take the 32-key chunks of the key set in turn, each with its own running (max, sum, output) per row; the
// partials are merged through shared memory at the end.  Lane j of a warp owns key j of the chunk during the logit
// phase and slice j of the output during the value phase.
template <typename T, int D, int R>
__global__ void __launch_bounds__(simt_warps(D) * 32) attn_simt_kernel(const SimtParams p) {
  constexpr int NW = simt_warps(D), NTH = NW * 32;
  constexpr int EPL = D / 32;
  constexpr int EPC = 16 / sizeof(T);                // elements per 16-byte load
  __shared__ __align__(16) float qs[R][D];
  __shared__ float part_o[NW][R][D];
  __shared__ float part_ml[NW][R][2];
  __shared__ int row_ok[R];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = (blockIdx.x / p.H) * R, h = blockIdx.x % p.H;
  const int nrows = p.q_rows ? min(*p.n_rows, p.rows_bound) : p.n_q;
  if (r0 >= nrows) return;
  if (threadIdx.x < R) {
    const int r = r0 + threadIdx.x;
    int ok = 0;
    if (r < nrows) {
      const int pos = p.q_rows ? p.q_rows[r] : p.q_base + r;
      ok = pos >= p.q_base && pos < p.q_base + p.n_q;
      if (!ok) set_status(p.status, FOCUS_ERR_INVALID_ARG);
    }
    row_ok[threadIdx.x] = ok;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < R * D; idx += NTH) {
    const int i = idx / D, c = idx % D;
    float v = 0.f;
    if (row_ok[i]) {
      const int pos = p.q_rows ? p.q_rows[r0 + i] : p.q_base + r0 + i;
      v = load_as_float((const T*)p.Q + (long long)(pos - p.q_base) * p.q_stride_row + (long long)h * p.q_stride_head + c);
    }
    qs[i][c] = v;
  }
  __syncthreads();
  const int g = h / p.hpg;
  const T* Kg = (const T*)p.K + (long long)g * p.kv_stride_head;
  const T* Vg = (const T*)p.V + (long long)g * p.kv_stride_head;
  const bool want_o = p.O != nullptr;
  float m[R], l[R], o[R][EPL];
#pragma unroll
  for (int i = 0; i < R; ++i) {
    m[i] = -INFINITY; l[i] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[i][e] = 0.f;
  }
  int chunk = 0;                                     // chunk counter, the same in every warp
  auto mine = [&]() { return (chunk++ % NW) == warp; };

  auto step = [&](int key) {
    float s[R];
#pragma unroll
    for (int i = 0; i < R; ++i) s[i] = 0.f;
    if (key >= 0) {
      const uint4* kr = reinterpret_cast<const uint4*>(Kg + (long long)key * p.kv_stride_tok);
#pragma unroll UNROLL_DOT
      for (int c = 0; c < D / EPC; ++c) {
        const uint4 raw = __ldg(kr + c);
        float kf[EPC];
        if constexpr (sizeof(T) == 2) {
          const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
          for (int e = 0; e < 4; ++e) { const float2 f = __bfloat1622float2(pb[e]); kf[2 * e] = f.x; kf[2 * e + 1] = f.y; }
        } else {
          kf[0] = __uint_as_float(raw.x); kf[1] = __uint_as_float(raw.y);
          kf[2] = __uint_as_float(raw.z); kf[3] = __uint_as_float(raw.w);
        }
#pragma unroll
        for (int i = 0; i < R; ++i) {
#pragma unroll
          for (int e4 = 0; e4 < EPC; e4 += 4) {
            const float4 q4 = *reinterpret_cast<const float4*>(&qs[i][c * EPC + e4]);   // same address in every lane
            s[i] = fmaf(q4.x, kf[e4], s[i]); s[i] = fmaf(q4.y, kf[e4 + 1], s[i]);
            s[i] = fmaf(q4.z, kf[e4 + 2], s[i]); s[i] = fmaf(q4.w, kf[e4 + 3], s[i]);
          }
        }
      }
    }
    // row maxima and row sums of the R rows as interleaved butterflies (R independent shuffles per level)
    float si[R], mx[R], pj[R], corr[R];
#pragma unroll
    for (int i = 0; i < R; ++i) { si[i] = key >= 0 ? s[i] * p.scale : -INFINITY; mx[i] = si[i]; }
#pragma unroll
    for (int ofs = 16; ofs > 0; ofs >>= 1) {
#pragma unroll
      for (int i = 0; i < R; ++i) mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], ofs));
    }
    bool any = false;
#pragma unroll
    for (int i = 0; i < R; ++i) {
      pj[i] = 0.f; corr[i] = 1.f;
      if (mx[i] != -INFINITY) {                      // warp-uniform
        any = true;
        const float m_new = fmaxf(m[i], mx[i]);
        corr[i] = expf(m[i] - m_new);
        pj[i] = key >= 0 ? expf(si[i] - m_new) : 0.f;
        m[i] = m_new;
      }
    }
    float ps[R];
#pragma unroll
    for (int i = 0; i < R; ++i) ps[i] = pj[i];
#pragma unroll
    for (int ofs = 16; ofs > 0; ofs >>= 1) {
#pragma unroll
      for (int i = 0; i < R; ++i) ps[i] += __shfl_xor_sync(0xffffffffu, ps[i], ofs);
    }
#pragma unroll
    for (int i = 0; i < R; ++i) {
      l[i] = l[i] * corr[i] + ps[i];
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[i][e] *= corr[i];
    }
    if (want_o && any) {
      // the 32 V rows of the chunk, sixteen loads in flight; an absent key reads row 0 and is discarded
#pragma unroll UNROLL_V
      for (int jj = 0; jj < 32; ++jj) {
        const int kk = __shfl_sync(0xffffffffu, key, jj);
        float v[EPL];
        load_slice<T, EPL>(Vg + (long long)max(kk, 0) * p.kv_stride_tok + lane * EPL, v);
#pragma unroll
        for (int e = 0; e < EPL; ++e) v[e] = kk >= 0 ? v[e] : 0.f;
#pragma unroll
        for (int i = 0; i < R; ++i) {
          const float pk = __shfl_sync(0xffffffffu, pj[i], jj);
#pragma unroll
          for (int e = 0; e < EPL; ++e) o[i][e] = fmaf(pk, v[e], o[i][e]);
        }
      }
    }
  };
  auto span = [&](int lo, int hi) {
    for (int j0 = lo; j0 < hi; j0 += 32)
      if (mine()) step(j0 + lane < hi ? j0 + lane : -1);
  };

  if (p.dense) {
    span(0, p.L);
  } else {
    const int row = g * p.group_stride;
    const int cnt = min(p.block_cnt[row], p.max_blocks);
    for (int bi = 0; bi < cnt; ++bi) {
      const int b = p.block_idx[(size_t)row * p.max_blocks + bi];
      if (b < 0 || b >= p.nb) {
        if (threadIdx.x == 0) set_status(p.status, FOCUS_ERR_INVALID_ARG);
        continue;
      }
      span(b * p.B, min((b + 1) * p.B, p.M));
    }
    for (int s0 = 0; s0 < p.n_sink; s0 += 32) {
      if (!mine()) continue;
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
  // merge of the warps' partials, warps in index order
#pragma unroll
  for (int i = 0; i < R; ++i) {
    if (lane == 0) { part_ml[warp][i][0] = m[i]; part_ml[warp][i][1] = l[i]; }
    if (want_o) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) part_o[warp][i][lane * EPL + e] = o[i][e];
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < R * D; idx += NTH) {
    const int i = idx / D, c = idx % D;
    if (!row_ok[i]) continue;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w)
      if (part_ml[w][i][1] > 0.f) mm = fmaxf(mm, part_ml[w][i][0]);
    float acc = 0.f, tot = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float wgt = part_ml[w][i][1] > 0.f ? expf(part_ml[w][i][0] - mm) : 0.f;
      tot += wgt * part_ml[w][i][1];
      if (want_o && wgt > 0.f) acc = fmaf(wgt, part_o[w][i][c], acc);
    }
    const int r = r0 + i;
    if (want_o) {
      const float outv = tot > 0.f ? acc / tot : 0.f;
      if constexpr (sizeof(T) == 2) ((__nv_bfloat16*)p.O)[((size_t)r * p.H + h) * D + c] = __float2bfloat16_rn(outv);
      else ((float*)p.O)[((size_t)r * p.H + h) * D + c] = outv;
    }
    if (p.lse && c == 0) p.lse[(size_t)h * p.lse_stride + r] = mm + logf(tot);
  }
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
  if (a.max_rows == 0) return FOCUS_OK;
  constexpr int R = 8;                               // query rows per CTA
  const unsigned grid = (unsigned)(((long long)a.max_rows + R - 1) / R * a.sh.n_q_heads);
  const bool bf = a.sh.dtype == FOCUS_BF16;
  if (a.sh.head_dim == 128) {
    if (bf) attn_simt_kernel<__nv_bfloat16, 128, R><<<grid, simt_warps(128) * 32, 0, st>>>(p);
    else attn_simt_kernel<float, 128, R><<<grid, simt_warps(128) * 32, 0, st>>>(p);
  } else {
    if (bf) attn_simt_kernel<__nv_bfloat16, 64, R><<<grid, simt_warps(64) * 32, 0, st>>>(p);
    else attn_simt_kernel<float, 64, R><<<grid, simt_warps(64) * 32, 0, st>>>(p);
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
