// Attention-sink column sums on the tensor cores (Eq. 6): part[h][j] = sum_i exp(scale * q_i^h . k_j - lse_i^h)
// over the active query rows i.  bf16 inputs, head_dim 128.
//
// The product is taken transposed, S^T = K_tile Q^T, so that TMEM lanes are keys and TMEM columns are query
// rows: each consumer thread owns one key and adds up its probabilities over the columns serially -- the
// column sum needs no cross-thread reduction and no second pass over the tile.  K streams once through a TMA
// ring (this kernel is HBM-bound); the query rows of one KV group stay resident in shared memory.
//
// Warp roles (320 threads): warp 0 TMA producer, warp 1 tcgen05.mma issuer + TMEM owner, warps 2..5 and 6..9 two
// consumer warpgroups that take the (key tile, head) units in turn: one warpgroup alone (a 64-column row of
// exponentials per thread and unit) was the slowest stage of the pipeline.
#include "tc_common.cuh"

using namespace tc;

namespace {

constexpr int TK = 128;               // keys per tile (MMA M)
constexpr int HD = 128;
constexpr int SLOT_BYTES = TK * HD * 2;
constexpr int HALF_BYTES = SLOT_BYTES / 2;
constexpr int NTHREADS = 320;
constexpr int MAX_SLOTS = 6;             // barrier slots laid out in shared memory
constexpr int RING_SLOTS = 4;            // K ring slots in use
constexpr int MAX_NPAD = 256;
constexpr int MAX_BUF = 8;              // TMEM accumulator buffers (512 columns / buffer width)

struct SinkParams {
  const __nv_bfloat16* Q;
  const int32_t* active_idx;
  const int32_t* n_active;
  const float* lse;             // [H][lse_stride], natural log
  float* part;                  // [H][L]
  long long q_stride_row, q_stride_head;
  int q_base, L, hpg, max_active, n_pad, n_slots, lse_stride, chunks;
  int n_buf, buf_cols;           // accumulator ring in TMEM: n_buf buffers of buf_cols columns
  int Hkv, n_ctas, groups_staged; // flat split of the Hkv*T key tiles over n_ctas CTAs; a CTA touches <= groups_staged heads
  int kv_div;                     // the kernel walks QUERY heads (Hkv = H, hpg = 1); query head h reads KV head h / kv_div
  float scale_log2;
  int32_t* status;
};


#define TC_LD16(taddr, r)                                                                                         \
  asm volatile(                                                                                                   \
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"     \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), \
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])                  \
      : "r"(taddr)                                                                                                \
      : "memory")

__global__ void __launch_bounds__(NTHREADS, 1)
sink_colsum_tc_kernel(const __grid_constant__ CUtensorMap tmK, const SinkParams p) {
  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // The Hkv * T key tiles (T per KV head) are cut into n_ctas contiguous ranges, one per CTA (one CTA per SM,
  // every SM busy); a range may cross from one KV head into the next, so the queries of both are staged.
  const int T = (p.L + TK - 1) / TK;
  const long long U = (long long)p.Hkv * T;
  const int u0 = (int)(U * blockIdx.x / p.n_ctas), u1 = (int)(U * (blockIdx.x + 1) / p.n_ctas);
  const int nt = u1 - u0;
  if (nt <= 0) return;
  const int g0 = u0 / T;
  const int ngs = min((u1 - 1) / T - g0 + 1, p.groups_staged);
  const int n = min(max(*p.n_active, 0), p.max_active);
  const int q_head_bytes = p.n_pad * 256;              // two swizzled halves of n_pad rows x 128 bytes
  const int q_bytes = p.groups_staged * p.hpg * q_head_bytes;

  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sptr = smem_raw + (sbase - smem_u32(smem_raw));
  const uint32_t sQ = sbase;
  const uint32_t sSlot = sbase + q_bytes;
  const uint32_t sBar = sSlot + p.n_slots * SLOT_BYTES;
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (MAX_SLOTS + s); };
  auto bar_sfull = [&](int b) { return sBar + 8u * (2 * MAX_SLOTS + b); };
  auto bar_sempty = [&](int b) { return sBar + 8u * (2 * MAX_SLOTS + MAX_BUF + b); };
  uint8_t* tail = sptr + q_bytes + p.n_slots * SLOT_BYTES + (2 * MAX_SLOTS + 2 * MAX_BUF) * 8;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4);
  float* neg_lse2 = reinterpret_cast<float*>(tail + 16);       // [staged heads][n_pad]: -lse * log2(e)

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.n_slots; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    for (int b = 0; b < p.n_buf; ++b) { mbar_init(bar_sfull(b), 1); mbar_init(bar_sempty(b), 128); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
    prefetch_tmap(&tmK);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_holder), 512);
    tmem_relinquish();
  }
  // query rows of every head of the staged group(s) -> swizzled K-major B operand; rows >= n are zero
  const int heads_staged = ngs * p.hpg;
  for (int idx = threadIdx.x; idx < heads_staged * p.n_pad * 16; idx += NTHREADS) {
    const int c = idx & 15, r = (idx >> 4) % p.n_pad, hs = (idx >> 4) / p.n_pad;     // hs = staged head slot
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < n) {
      const int pos = p.active_idx[r];
      if (pos >= p.q_base && pos < p.L) {
        v = __ldg(reinterpret_cast<const uint4*>(p.Q + (long long)(pos - p.q_base) * p.q_stride_row +
                                                 (long long)(g0 * p.hpg + hs) * p.q_stride_head + c * 8));
      } else if (c == 0) {
        set_status(p.status, FOCUS_ERR_INVALID_ARG);
      }
    }
    const int half = c >> 3, cc = c & 7;
    *reinterpret_cast<uint4*>(sptr + hs * q_head_bytes + half * (p.n_pad * 128) + r * 128 + ((cc ^ (r & 7)) << 4)) = v;
  }
  for (int idx = threadIdx.x; idx < heads_staged * p.n_pad; idx += NTHREADS) {
    const int r = idx % p.n_pad, hs = idx / p.n_pad;
    neg_lse2[idx] = r < n ? -p.lse[(size_t)(g0 * p.hpg + hs) * p.lse_stride + r] * 1.4426950408889634f : -INFINITY;
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_holder;
  const int units = nt * p.hpg;                  // one unit = (key tile, query head of the group)
  const int ncol = max(32, (n + 31) & ~31);       // query columns in use: the active rows, padded to 32 (one TMEM load)

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      // tile t of head g; ring slot and phase follow the tile counter without divisions
      const uint64_t l2_pol = l2_policy_evict_first();      // K streams through once: do not keep it in L2
      int t = u0 % T, g = u0 / T, kvh = g / p.kv_div, slot = 0;
      uint32_t ph = 0;
      for (int i = 0; i < nt && ok; ++i) {
        if (!mbar_wait(bar_empty(slot), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
        const uint32_t dst = sSlot + slot * SLOT_BYTES;
        mbar_expect_tx(bar_full(slot), SLOT_BYTES);
        tma_load_3d_hint(dst, &tmK, bar_full(slot), 0, t * TK, kvh, l2_pol);
        tma_load_3d_hint(dst + HALF_BYTES, &tmK, bar_full(slot), 64, t * TK, kvh, l2_pol);
        ++issued;
        if (++slot == p.n_slots) { slot = 0; ph ^= 1u; }
        if (++t == T) { t = 0; ++g; kvh = g / p.kv_div; }
      }
      if (!ok) {
        const int first = issued > p.n_slots ? issued - p.n_slots : 0;
        for (int i = first; i < issued; ++i) {
          const uint64_t t_start = global_ns();
          while (!mbar_try_wait(bar_full(i % p.n_slots), (uint32_t)(i / p.n_slots) & 1u))
            if (global_ns() - t_start > WAIT_LIMIT_NS) break;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(TK, ncol, 0);
      bool ok = true;
      // unit u = (key tile i, head hh of the group); slot/phase of the K ring, buffer/phase of the accumulator ring
      // and the staged head slot follow u without divisions
      const int nbuf_mask = p.n_buf - 1, nbuf_shift = 31 - __clz(p.n_buf);
      int hh = 0, slot = 0, t = u0 % T, hs0 = (u0 / T - g0) * p.hpg;
      uint32_t ph = 0;
      for (int u = 0; u < units && ok; ++u) {
        const int b = u & nbuf_mask;
        if (!mbar_wait(bar_sempty(b), ((uint32_t)(u >> nbuf_shift) & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
        if (hh == 0 && !mbar_wait(bar_full(slot), ph, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint64_t kdesc = make_sdesc(sSlot + slot * SLOT_BYTES, 16, 1024);
        const uint64_t qdesc = make_sdesc(sQ + (hs0 + hh) * q_head_bytes, 16, 1024);
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            mma_ss(tmem + b * p.buf_cols, kdesc + (uint64_t)((half * HALF_BYTES + ks * 32) >> 4),
                   qdesc + (uint64_t)((half * (p.n_pad * 128) + ks * 32) >> 4), idesc, (half | ks) ? 1u : 0u);
        tc_commit(bar_sfull(b));
        if (++hh == p.hpg) {
          hh = 0;
          tc_commit(bar_empty(slot));
          if (++slot == p.n_slots) { slot = 0; ph ^= 1u; }
          if (++t == T) { t = 0; hs0 += p.hpg; }
        }
      }
    }
  } else {
    const int rq = warp & 3;                                  // TMEM lane quarter this warp may access
    const int krow = rq * 32 + lane;                          // key of this thread inside the tile
    const uint32_t lane_off = (uint32_t)(rq * 32) << 16;
    // unit u = (key tile i = u / hpg, head hh = u % hpg of the group); the counters below follow u without divisions
    const int cw = (warp - 2) >> 2;                           // consumer warpgroup: units cw, cw + 2, ...
    const int nbuf_mask = p.n_buf - 1, nbuf_shift = 31 - __clz(p.n_buf);   // n_buf is a power of two (2, 4 or 8)
    int i = cw / p.hpg, hh = cw % p.hpg;
    int t = (u0 + i) % T, g = (u0 + i) / T;
    for (int u = cw; u < units; u += 2) {
      const int b = u & nbuf_mask;
      if (!__all_sync(0xffffffffu, mbar_wait(bar_sfull(b), (uint32_t)(u >> nbuf_shift) & 1u, abort_flag, p.status))) break;
      tc_fence_after();
      const float* nl = neg_lse2 + ((g - g0) * p.hpg + hh) * p.n_pad;
      float acc = 0.f;
      const uint32_t tsrc = tmem + lane_off + b * p.buf_cols;
      // columns in groups of 64: both 32-column loads of a group are requested before the single wait; the
      // accumulator buffer goes back to the MMA warp as soon as its last group sits in registers.  Columns past
      // the n active rows carry -inf in nl[] (their probabilities are zero).
      float acc4[4] = {0.f, 0.f, 0.f, 0.f};
      for (int c0 = 0; c0 < ncol; c0 += 64) {
        uint32_t r[64];
        const bool two = c0 + 32 < ncol;
        TC_LD32(tsrc + c0, (r + 0));
        if (two) TC_LD32(tsrc + c0 + 32, (r + 32));
        tc_wait_ld();
        if (c0 + 64 >= ncol) {
          tc_fence_before();
          mbar_arrive(bar_sempty(b));
        }
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          if (hf == 0 || two) {
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
              const float4 nv = *reinterpret_cast<const float4*>(nl + c0 + hf * 32 + c4 * 4);
              acc4[0] += ex2(fmaf(__uint_as_float(r[hf * 32 + c4 * 4 + 0]), p.scale_log2, nv.x));
              acc4[1] += ex2(fmaf(__uint_as_float(r[hf * 32 + c4 * 4 + 1]), p.scale_log2, nv.y));
              acc4[2] += ex2(fmaf(__uint_as_float(r[hf * 32 + c4 * 4 + 2]), p.scale_log2, nv.z));
              acc4[3] += ex2(fmaf(__uint_as_float(r[hf * 32 + c4 * 4 + 3]), p.scale_log2, nv.w));
            }
          }
        }
      }
      acc = (acc4[0] + acc4[1]) + (acc4[2] + acc4[3]);
      const int key = t * TK + krow;
      if (key < p.L) p.part[(size_t)(g * p.hpg + hh) * p.L + key] = acc;
      hh += 2;
      while (hh >= p.hpg) {
        hh -= p.hpg;
        if (++t == T) { t = 0; ++g; }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

static int sink_npad(int max_active) { return (max_active + 31) / 32 * 32; }
static int sink_slots(int heads_staged, int n_pad) {
  const int fixed = 1024 + heads_staged * n_pad * 256 + (2 * MAX_SLOTS + 2 * MAX_BUF) * 8 + 16 + heads_staged * n_pad * 4 + 64;
  int s = (232448 - fixed) / SLOT_BYTES;
  // more copies in flight per CTA only share the CTA's bandwidth among themselves: the tile needed next lands later
  // (measured at 32K, 32 heads: the whole call 71.4 us with six slots, 69.3 with four)
  return s > RING_SLOTS ? RING_SLOTS : s;
}

bool sink_tc_supported(const focus_ctx* ctx, const focus_shape* s, int max_active) {
  if (!ctx->encode_tiled || s->dtype != FOCUS_BF16 || s->head_dim != HD) return false;
  const int n_pad = sink_npad(max_active);
  return n_pad <= MAX_NPAD && sink_slots(1, n_pad) >= 2;
}

focus_status launch_sink_colsum_tc(focus_ctx* ctx, const focus_shape* s, const void* Q, int q_base,
                                   const int32_t* active_idx, const int32_t* n_active, int max_active, const void* K,
                                   const float* lse, float* part, WsAlloc&, cudaStream_t st) {
  // Every query head is walked on its own (its key tiles come from KV head h / (H / Hkv)): with GQA the K tiles of
  // a KV head are then read once per query head of the group, from L2 after the first, but a CTA stages the
  // queries of at most two heads instead of two whole groups.
  const int kvh = s->n_kv_heads, H = s->n_q_heads;
  const int Hkv = H, hpg = 1;
  SinkParams p;
  p.kv_div = H / kvh;
  p.Q = (const __nv_bfloat16*)Q; p.active_idx = active_idx; p.n_active = n_active; p.lse = lse; p.part = part;
  p.q_stride_row = s->q_stride_row; p.q_stride_head = s->q_stride_head;
  p.q_base = q_base; p.L = s->L; p.hpg = hpg; p.max_active = max_active; p.n_pad = sink_npad(max_active);
  p.lse_stride = max_active;
  p.buf_cols = p.n_pad <= 64 ? 64 : (p.n_pad <= 128 ? 128 : 256);
  p.n_buf = 512 / p.buf_cols;
  const int T = (s->L + TK - 1) / TK;
  // one CTA per SM over the flat tile range when the queries of two KV heads fit beside >= 4 ring slots and no
  // range can span more than two heads; otherwise whole chunks of single heads
  p.Hkv = Hkv;
  const long long U = (long long)Hkv * T;
  if (sink_slots(2 * hpg, p.n_pad) >= 4 && U / ctx->sm_count + 1 <= T && U >= ctx->sm_count) {
    p.groups_staged = 2;
    p.n_ctas = ctx->sm_count;
  } else {
    p.groups_staged = 1;
    int chunks = ctx->sm_count / Hkv;
    if (chunks < 1) chunks = 1;
    if (chunks > T) chunks = T;
    p.n_ctas = chunks * Hkv;            // ranges of T / chunks tiles never cross a head when chunks divides evenly...
    while (T % chunks) --chunks;        // ...so take a divisor of T
    p.n_ctas = chunks * Hkv;
  }
  p.chunks = 0;
  p.n_slots = sink_slots(p.groups_staged * hpg, p.n_pad);
  p.scale_log2 = shape_scale(s) * 1.4426950408889634f;
  p.status = ctx->d_status;
  CUtensorMap tmK;
  if (!encode_kv_map(ctx->encode_tiled, &tmK, K, HD, s->L, kvh, s->kv_stride_tok, s->kv_stride_head, 64, TK))
    return FOCUS_ERR_INVALID_ARG;
  const int hs = p.groups_staged * hpg;
  const int smem = 1024 + hs * p.n_pad * 256 + p.n_slots * SLOT_BYTES + (2 * MAX_SLOTS + 2 * MAX_BUF) * 8 + 16 +
                   hs * p.n_pad * 4 + 64;
  int& attr_smem = ctx->ls.sink_attr_smem;
  if (smem > attr_smem) {
    if (cudaFuncSetAttribute(sink_colsum_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return FOCUS_ERR_CUDA;
    attr_smem = smem;
  }
  sink_colsum_tc_kernel<<<p.n_ctas, NTHREADS, smem, st>>>(tmK, p);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}
