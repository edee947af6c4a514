// One sparse layer in two launches (Algorithm 1, sparse branch): a fused selection kernel (block relevance against
// the cached pooled keys, Top-C, sink keep flags, column mask, sink row gather) and the block-sparse attention
// kernel (split merge included), chained by programmatic dependent launch.  The stand-alone entry points compute
// the same quantities one launch per stage.
#include "focus_common.cuh"

constexpr int FS_THREADS = 1024;
constexpr int FS_MAX_NB = 8192;
constexpr int FS_HD = 128;

// CTAs [0, Hkv): selection for KV head g.  CTAs [Hkv, ...): gather 64 sink rows of K and V of one KV head each.
// At most 32 registers per thread: two CTAs fit one SM, so the selection CTAs of all KV heads can run on the SMs
// that an attention launch of 128 CTAs leaves idle, ahead of the dependency wait.
__global__ void __launch_bounds__(FS_THREADS, 2)
fused_select_kernel(const __nv_bfloat16* __restrict__ Q, int q_base, long long q_stride_row, long long q_stride_head,
                    const int32_t* __restrict__ focus_idx, const int32_t* __restrict__ n_focus, int max_focus,
                    const float* __restrict__ Kbar, int Hkv, int hpg, int L, int M, int B, int nb, int C,
                    const int32_t* __restrict__ sink_idx, int n_sink, int ns_pad,
                    const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V, long long kv_stride_tok,
                    long long kv_stride_head, float* __restrict__ R, int32_t* __restrict__ block_idx,
                    int32_t* __restrict__ block_cnt, uint8_t* __restrict__ sink_keep, __nv_bfloat16* __restrict__ gK,
                    __nv_bfloat16* __restrict__ gV, uint8_t* __restrict__ mask, int32_t* status) {
  const int tid = threadIdx.x;
  // The attention kernel of this layer is launched as a programmatic dependent: let its CTAs start their own
  // set-up now; it waits for this grid to complete before it reads anything written here.  This kernel may itself
  // have been started before its predecessor in the stream finished.  The only kernels that let a successor start
  // early are this one and the attention kernels; what they may still be reading are the buffers written below
  // after griddepcontrol.wait (block list and count, keep flags, mask, gathered rows).  Everything read before the
  // wait (Q, pooled keys, K/V rows, focus and sink indices) comes from kernels that do not release their successors
  // early, so it is complete once this kernel runs at all; R and the status word are read by no such kernel.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if ((int)blockIdx.x >= Hkv) {
    // ---- gather: 64 sink rows of one KV head per CTA, one 16-byte chunk of K and of V per thread ---------
    const int gi = (int)blockIdx.x - Hkv;
    const int g = gi % Hkv;
    const int s = (gi / Hkv) * 64 + (tid >> 4), c = tid & 15;
    if (s >= ns_pad) return;
    uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
    if (s < n_sink) {
      const int j = sink_idx[s];
      if (j < 0 || j >= L) {
        if (c == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
      } else {
        const size_t off = (size_t)g * kv_stride_head + (size_t)j * kv_stride_tok + c * 8;
        kv = __ldg(reinterpret_cast<const uint4*>(K + off));
        vv = __ldg(reinterpret_cast<const uint4*>(V + off));
      }
    }
    const size_t o = ((size_t)g * ns_pad + s) * FS_HD + c * 8;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    *reinterpret_cast<uint4*>(gK + o) = kv;
    *reinterpret_cast<uint4*>(gV + o) = vv;
    return;
  }
  // ---- selection for KV head g -------------------------------------------------------------------------
  __shared__ uint32_t key[FS_MAX_NB];
  __shared__ uint8_t sel[FS_MAX_NB];
  __shared__ float part[8][FS_HD];
  __shared__ float qbar[FS_HD];
  __shared__ int scan_s[33];
  __shared__ int hist[258];
  const int g = blockIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  // Issue every load that does not depend on another one first: the kernel is a chain of global-memory
  // latencies, not of bandwidth.
  constexpr int KPRE = 4;
  const float* kb = Kbar + (size_t)g * nb * FS_HD + lane * 4;
  float4 kpre[KPRE];
#pragma unroll
  for (int u = 0; u < KPRE; ++u) {
    const int b = warp + u * (FS_THREADS / 32);
    kpre[u] = b < nb ? __ldg(reinterpret_cast<const float4*>(kb + (size_t)b * FS_HD)) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const int my_sink = tid < n_sink ? sink_idx[tid] : -1;
  // The gather CTAs of this launch mostly run only after the previous attention launch has left the SMs: bring the
  // sink rows of this head into L2 now, while that launch is still streaming, so that they find them there.
  for (int s = tid; s < n_sink; s += FS_THREADS) {
    const int j = s == tid ? my_sink : sink_idx[s];
    if (j >= 0 && j < L) {
      const size_t off = (size_t)g * kv_stride_head + (size_t)j * kv_stride_tok;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(K + off));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(K + off + 64));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(V + off));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(V + off + 64));
    }
  }
  const int c = tid & 127, y = tid >> 7;
  const int pos0 = y < max_focus ? focus_idx[y] : -1;
  const int nf = min(max(*n_focus, 0), max_focus);
  {
    float acc = 0.f;
    for (int i = y; i < nf; i += 8) {
      const int pos = i == y ? pos0 : focus_idx[i];
      if (pos < q_base || pos >= L) {
        if (c == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
        continue;
      }
      const __nv_bfloat16* row = Q + (long long)(pos - q_base) * q_stride_row + (long long)(g * hpg) * q_stride_head + c;
      for (int hh = 0; hh < hpg; ++hh) acc += __bfloat162float(row[(long long)hh * q_stride_head]);
    }
    part[y][c] = acc;
  }
  __syncthreads();
  if (tid < FS_HD) {
    float s = 0.f;
#pragma unroll
    for (int yy = 0; yy < 8; ++yy) s += part[yy][tid];
    qbar[tid] = nf > 0 ? s / (float)(nf * hpg) : 0.f;
    if (tid == 0 && nf == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
  }
  __syncthreads();
  {
    const float4 qv = *reinterpret_cast<const float4*>(&qbar[lane * 4]);
    auto score = [&](int b, const float4& kv) {
      float s = kv.x * qv.x + kv.y * qv.y + kv.z * qv.z + kv.w * qv.w;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) key[b] = float_key(s);             // R itself is written after the dependency wait, from the key
    };
#pragma unroll
    for (int u = 0; u < KPRE; ++u) {
      const int b = warp + u * (FS_THREADS / 32);
      if (b < nb) score(b, kpre[u]);
    }
#pragma unroll 4
    for (int b = warp + KPRE * (FS_THREADS / 32); b < nb; b += FS_THREADS / 32)
      score(b, __ldg(reinterpret_cast<const float4*>(kb + (size_t)b * FS_HD)));
  }
  __syncthreads();
  if (nb <= 256) {                                   // few blocks: rank by counting, one pass, no histogram
    for (int i = tid; i < nb; i += FS_THREADS) {
      const uint32_t ki = key[i];
      int rank = 0;
      for (int j = 0; j < nb; ++j) {
        const uint32_t kj = key[j];
        rank += (kj > ki || (kj == ki && j < i)) ? 1 : 0;
      }
      sel[i] = rank < C;
    }
    __syncthreads();
  } else {
    block_topc_mark(key, nb, C, sel, hist, scan_s);
  }
  // Everything that can be computed ahead of the dependency wait is: with at most one block and one sink slot per
  // thread (every benchmark shape) the list position of this thread's block and the flags of its sink token sit in
  // registers, and what follows the wait is a handful of independent stores, no loop, no barrier.
  const bool one_pass = nb <= FS_THREADS && ns_pad <= FS_THREADS;
  int my_f = 0, my_posn = 0, base = 0;
  uint8_t my_keep = 0, my_mk = 0;
  if (one_pass) {
    my_f = (tid < nb && sel[tid]) ? 1 : 0;
    my_posn = block_excl_scan(my_f, scan_s, base);
    if (tid < n_sink && my_sink >= 0 && my_sink < L) {
      const int b = my_sink / B;
      my_keep = (b < nb && !sel[b]) ? 1 : 0;
      my_mk = (my_keep && my_sink < M) ? 1 : 0;
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // every store comes after the wait: the previous layer's selection kernel (which may still have been storing when
  // this one started) wrote the same R, lists and flags
  int32_t* out = block_idx + (size_t)g * C;
  if (one_pass) {
    if (R && tid < nb) R[(size_t)g * nb + tid] = key_to_float(key[tid]);
    if (tid < ns_pad) {
      if (tid < n_sink && sink_keep) sink_keep[(size_t)g * n_sink + tid] = my_keep;
      mask[(size_t)g * ns_pad + tid] = my_mk;
    }
    if (my_f && my_posn < C) out[my_posn] = tid;
  } else {
    if (R)
      for (int b = tid; b < nb; b += FS_THREADS) R[(size_t)g * nb + b] = key_to_float(key[b]);
    for (int s = tid; s < ns_pad; s += FS_THREADS) {
      uint8_t keep = 0, mk = 0;
      if (s < n_sink) {
        const int j = s == tid ? my_sink : sink_idx[s];
        if (j >= 0 && j < L) {
          const int b = j / B;
          keep = (b < nb && !sel[b]) ? 1 : 0;
          mk = (keep && j < M) ? 1 : 0;
        }
        if (sink_keep) sink_keep[(size_t)g * n_sink + s] = keep;
      }
      mask[(size_t)g * ns_pad + s] = mk;
    }
    base = 0;
    for (int c0 = 0; c0 < nb; c0 += FS_THREADS) {
      const int i = c0 + tid;
      const int f = (i < nb && sel[i]) ? 1 : 0;
      int tot;
      const int pre = block_excl_scan(f, scan_s, tot);
      if (f && base + pre < C) out[base + pre] = i;
      base += tot;
    }
  }
  if (tid == 0) block_cnt[g] = min(base, C);
}

extern "C" focus_status focus_sparse_layer(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base,
                                           int32_t n_q, const int32_t* q_rows, const int32_t* n_rows, int32_t max_rows,
                                           const int32_t* focus_idx, const int32_t* n_focus, int32_t max_focus,
                                           const void* K, const void* V, const float* Kbar, int32_t C,
                                           const int32_t* sink_idx, int32_t n_sink, float* R, int32_t* block_idx,
                                           int32_t* block_cnt, uint8_t* sink_keep, void* O, float* lse,
                                           focus_stream stream) {
  FOCUS_STAGE("focus_sparse_layer");
  if (!ctx || !shape_ok_basic(shape) || !Q || !K || !V || !Kbar || !O || !focus_idx || !n_focus || !block_idx ||
      !block_cnt)
    return FOCUS_ERR_INVALID_ARG;
  if (!all_aligned16(Q, K, V, Kbar, O)) return FOCUS_ERR_INVALID_ARG;
  const int nb = shape_nb(shape);
  if (C < 0 || C > nb || n_sink < 0 || max_focus <= 0) return FOCUS_ERR_INVALID_ARG;
  if (n_sink > 0 && (!sink_idx || !sink_keep)) return FOCUS_ERR_INVALID_ARG;
  if (n_q < 0 || q_base < 0 || q_base + n_q > shape->L) return FOCUS_ERR_INVALID_ARG;
  if ((q_rows == nullptr) != (n_rows == nullptr) || (q_rows && max_rows < 0)) return FOCUS_ERR_INVALID_ARG;
  if (!shape_supported(shape)) return FOCUS_ERR_UNSUPPORTED;

  AttnArgs a{};
  a.sh = *shape; a.scale = shape_scale(shape);
  a.Q = Q; a.q_base = q_base; a.n_q = n_q; a.q_rows = q_rows; a.n_rows = n_rows;
  a.max_rows = q_rows ? max_rows : n_q;
  a.K = K; a.V = V; a.O = O; a.lse = lse; a.lse_stride = a.max_rows;
  a.dense = 0; a.group_stride = 1; a.block_idx = block_idx; a.max_blocks = C; a.block_cnt = block_cnt;
  a.sink_idx = sink_idx; a.sink_keep = sink_keep; a.n_sink = n_sink;

  const bool fused = !ctx->force_simt && attn_tc_supported(ctx, a) && shape->head_dim == FS_HD && nb <= FS_MAX_NB &&
                     nb > 0 && a.max_rows > 0;
  if (!fused) {
    // generic route: the stand-alone stages, one after the other
    if (!R) return FOCUS_ERR_INVALID_ARG;
    focus_status s = focus_score_blocks(ctx, shape, Q, q_base, focus_idx, n_focus, max_focus, nullptr, Kbar,
                                        FOCUS_HEADS_PER_KV_GROUP, R, stream);
    if (s != FOCUS_OK) return s;
    s = focus_select_blocks(ctx, shape, R, FOCUS_HEADS_PER_KV_GROUP, C, sink_idx, n_sink, FOCUS_SINK_TOKENS, block_idx,
                            C, block_cnt, sink_keep, stream);
    if (s != FOCUS_OK) return s;
    return focus_sparse_attn(ctx, shape, Q, q_base, n_q, q_rows, n_rows, max_rows, K, V, FOCUS_HEADS_PER_KV_GROUP,
                             block_idx, C, block_cnt, sink_idx, sink_keep, n_sink, O, lse, stream);
  }
  const int Hkv = shape->n_kv_heads, hpg = shape->n_q_heads / Hkv;
  const int ns_pad = (n_sink + 127) / 128 * 128;
  WsAlloc ws(ctx);
  SinkGather sg{nullptr, nullptr, nullptr};
  if (ns_pad > 0) {
    sg.gK = ws.get<__nv_bfloat16>((size_t)Hkv * ns_pad * FS_HD);
    sg.gV = ws.get<__nv_bfloat16>((size_t)Hkv * ns_pad * FS_HD);
    sg.mask = ws.get<uint8_t>((size_t)Hkv * ns_pad);
  } else {
    sg.mask = ws.get<uint8_t>(256);
  }
  if (!ws.ok) return FOCUS_ERR_WORKSPACE_TOO_SMALL;
  const int grid = Hkv + (ns_pad + 63) / 64 * Hkv;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1); cfg.blockDim = dim3(FS_THREADS, 1, 1); cfg.dynamicSmemBytes = 0; cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = ctx->no_pdl ? 0 : 1;
  if (cudaLaunchKernelEx(&cfg, fused_select_kernel,
      (const __nv_bfloat16*)Q, q_base, (long long)shape->q_stride_row, (long long)shape->q_stride_head, focus_idx, n_focus,
      max_focus, Kbar, Hkv, hpg, (int)shape->L, (int)shape->M, (int)shape->kv_block, nb, C, sink_idx, n_sink, ns_pad,
      (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, (long long)shape->kv_stride_tok, (long long)shape->kv_stride_head, R,
      block_idx, block_cnt, sink_keep, sg.gK, sg.gV, sg.mask, ctx->d_status) != cudaSuccess) {
    cudaGetLastError();
    return FOCUS_ERR_CUDA;
  }
  FOCUS_CHECK_LAUNCH();
  return launch_attn_tc_ws(ctx, a, ws, &sg, stream);
}
