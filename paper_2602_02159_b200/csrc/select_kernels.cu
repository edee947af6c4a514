// Index-set selection kernels: past-confidence indicator + window expansion (Eq. 4, Eq. 5), Top-C block
// selection (Eq. 8) and Top-N_sink token selection (Section "Dynamic attention sinks identification").
// All three are comparison-only: scores are mapped to order-preserving integer keys, ties go to the
// lower index, outputs come out ascending through a block-wide prefix sum.
#include "focus_common.cuh"

// ------------------------------------------------------------------------------------------------
// Stage 1.  One CTA.  Candidates = masked positions of [blk_lo, blk_hi); rank by counting.
// ------------------------------------------------------------------------------------------------
constexpr int SQ_THREADS = 256;
constexpr int SQ_MAX_RANGE = 4096;
constexpr int SQ_MAX_K = 1024;

__global__ void __launch_bounds__(SQ_THREADS)
select_queries_kernel(const float* __restrict__ conf, const uint8_t* __restrict__ masked, int blk_lo, int blk_hi,
                      int k, int hw, int clip_lo, int clip_hi, int32_t* __restrict__ focus_idx,
                      int32_t* __restrict__ n_focus, int32_t* __restrict__ active_idx, int32_t* __restrict__ n_active) {
  __shared__ uint32_t key[SQ_MAX_RANGE];     // small ranges: key of every position; long ranges: keys of the candidates only
  __shared__ uint16_t cpos[SQ_MAX_RANGE];    // long ranges: position (relative to blk_lo) of the c-th candidate
  __shared__ uint8_t valid[SQ_MAX_RANGE];    // small ranges: masked flag; long ranges: selection flag of the c-th candidate
  __shared__ uint8_t sel[SQ_MAX_RANGE];
  __shared__ int focus_s[SQ_MAX_K];
  __shared__ int scan_s[33];
  __shared__ int hist[258];
  const int n = blk_hi - blk_lo;
  const int tid = threadIdx.x;
  if (n <= 256) {
    // rank by counting: one pass, quadratic in the range
    for (int i = tid; i < n; i += SQ_THREADS) {
      key[i] = float_key(conf[blk_lo + i]);
      valid[i] = masked[blk_lo + i] != 0;
    }
    __syncthreads();
    for (int i = tid; i < n; i += SQ_THREADS) {
      int rank = 0;
      if (valid[i]) {
        const uint32_t ki = key[i];
        for (int j = 0; j < n; ++j) {
          const uint32_t kj = key[j];
          rank += (valid[j] && (kj > ki || (kj == ki && j < i))) ? 1 : 0;
        }
      }
      sel[i] = valid[i] && rank < k;
    }
    __syncthreads();
  } else {
    // long ranges: the masked positions are compacted (index order kept), the k largest of their keys are marked by
    // the radix descent (equal keys in index order), and the marks are scattered back
    int n_cand = 0;
    for (int c0 = 0; c0 < n; c0 += SQ_THREADS) {
      const int i = c0 + tid;
      const int f = (i < n && masked[blk_lo + i] != 0) ? 1 : 0;
      int tot;
      const int pre = block_excl_scan(f, scan_s, tot);
      if (f) { key[n_cand + pre] = float_key(conf[blk_lo + i]); cpos[n_cand + pre] = (uint16_t)i; }
      if (i < n) sel[i] = 0;
      n_cand += tot;
    }
    __syncthreads();
    block_topc_mark(key, n_cand, min(k, n_cand), valid, hist, scan_s);
    for (int c = tid; c < n_cand; c += SQ_THREADS)
      if (valid[c]) sel[cpos[c]] = 1;
    __syncthreads();
  }
  // ascending compaction of the selected positions
  int base = 0;
  for (int c0 = 0; c0 < n; c0 += SQ_THREADS) {
    const int i = c0 + tid;
    const int f = (i < n && sel[i]) ? 1 : 0;
    int tot;
    const int pre = block_excl_scan(f, scan_s, tot);
    if (f) {
      focus_s[base + pre] = blk_lo + i;
      focus_idx[base + pre] = blk_lo + i;
    }
    base += tot;
  }
  const int nf = base;                       // = min(k, #candidates)
  for (int i = nf + tid; i < k; i += SQ_THREADS) focus_idx[i] = -1;
  if (tid == 0) *n_focus = nf;
  __syncthreads();
  // windows: pick i contributes the part of [f_i - hw, f_i + hw] not already covered by pick i-1
  const int span = 2 * hw + 1;
  int abase = 0;
  for (int c0 = 0; c0 < nf; c0 += SQ_THREADS) {
    const int i = c0 + tid;
    int lo = 0, cnt = 0;
    if (i < nf) {
      const int f = focus_s[i];
      lo = max(f - hw, clip_lo);
      if (i > 0) lo = max(lo, focus_s[i - 1] + hw + 1);
      const int hi = min(f + hw, clip_hi - 1);
      cnt = max(0, hi - lo + 1);
    }
    int tot;
    const int pre = block_excl_scan(cnt, scan_s, tot);
    for (int t = 0; t < cnt; ++t) active_idx[abase + pre + t] = lo + t;
    abase += tot;
  }
  for (int i = abase + tid; i < k * span; i += SQ_THREADS) active_idx[i] = -1;
  if (tid == 0) *n_active = abase;
  publish_outputs();
}

extern "C" focus_status focus_select_queries(focus_ctx* ctx, const float* conf_prev, const uint8_t* masked, int32_t L,
                                             int32_t blk_lo, int32_t blk_hi, int32_t k, int32_t w, int32_t clip_lo,
                                             int32_t clip_hi, int32_t* focus_idx, int32_t* n_focus,
                                             int32_t* active_idx, int32_t* n_active, focus_stream stream) {
  FOCUS_STAGE("focus_select_queries");
  if (!ctx || !conf_prev || !masked || !focus_idx || !n_focus || !active_idx || !n_active) return FOCUS_ERR_INVALID_ARG;
  if (L <= 0 || blk_lo < 0 || blk_hi < blk_lo || blk_hi > L || k < 0 || w < 0) return FOCUS_ERR_INVALID_ARG;
  if (clip_lo < 0 || clip_hi > L || clip_hi < clip_lo) return FOCUS_ERR_INVALID_ARG;
  if (blk_hi - blk_lo > SQ_MAX_RANGE || k > SQ_MAX_K) return FOCUS_ERR_UNSUPPORTED;
  select_queries_kernel<<<1, SQ_THREADS, 0, stream>>>(conf_prev, masked, blk_lo, blk_hi, k, w / 2, clip_lo, clip_hi,
                                                      focus_idx, n_focus, active_idx, n_active);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}

// ------------------------------------------------------------------------------------------------
// Stage 3b.  One CTA per group: rank-by-counting Top-C over nb <= 8192 block scores.
// ------------------------------------------------------------------------------------------------
constexpr int SB_THREADS = 1024;
constexpr int SB_MAX_NB = 8192;

__global__ void __launch_bounds__(SB_THREADS)
select_blocks_kernel(const float* __restrict__ R, int nb, int C, int B, const int32_t* __restrict__ sink_idx,
                     int n_sink, int sink_blocks_mode, int32_t* __restrict__ block_idx, int max_blocks,
                     int32_t* __restrict__ block_cnt, uint8_t* __restrict__ sink_keep, int32_t* status) {
  __shared__ uint32_t key[SB_MAX_NB];
  __shared__ uint8_t sel[SB_MAX_NB];
  __shared__ int scan_s[33];
  __shared__ int hist[258];
  const int g = blockIdx.x, tid = threadIdx.x;
  const float* Rg = R + (size_t)g * nb;
  for (int i = tid; i < nb; i += SB_THREADS) key[i] = float_key(Rg[i]);
  __syncthreads();
  if (nb <= 256) {                                   // few blocks: rank by counting, one pass, no histogram
    for (int i = tid; i < nb; i += SB_THREADS) {
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
  for (int s = tid; s < n_sink; s += SB_THREADS) {
    const int j = sink_idx[s];
    const int b = j / B;
    if (j < 0 || b >= nb) {
      set_status(status, FOCUS_ERR_INVALID_ARG);
      if (sink_keep) sink_keep[(size_t)g * n_sink + s] = 0;
      continue;
    }
    if (sink_blocks_mode) {
      sel[b] = 1;                                   // benign race: every writer stores 1
      if (sink_keep) sink_keep[(size_t)g * n_sink + s] = 0;
    } else {
      sink_keep[(size_t)g * n_sink + s] = sel[b] ? 0 : 1;
    }
  }
  __syncthreads();
  int base = 0;
  int32_t* out = block_idx + (size_t)g * max_blocks;
  for (int c0 = 0; c0 < nb; c0 += SB_THREADS) {
    const int i = c0 + tid;
    const int f = (i < nb && sel[i]) ? 1 : 0;
    int tot;
    const int pre = block_excl_scan(f, scan_s, tot);
    if (f && base + pre < max_blocks) out[base + pre] = i;
    base += tot;
  }
  if (base > max_blocks) {
    if (tid == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
    base = max_blocks;
  }
  for (int i = base + tid; i < max_blocks; i += SB_THREADS) out[i] = -1;
  if (tid == 0) block_cnt[g] = base;
}

extern "C" focus_status focus_select_blocks(focus_ctx* ctx, const focus_shape* shape, const float* R,
                                            int32_t head_reduce, int32_t C, const int32_t* sink_idx, int32_t n_sink,
                                            int32_t sink_mode, int32_t* block_idx, int32_t max_blocks,
                                            int32_t* block_cnt, uint8_t* sink_keep, focus_stream stream) {
  FOCUS_STAGE("focus_select_blocks");
  if (!ctx || !shape_ok_basic(shape) || !R || !block_idx || !block_cnt) return FOCUS_ERR_INVALID_ARG;
  const int nb = shape_nb(shape);
  if (C < 0 || C > nb || max_blocks < C || n_sink < 0) return FOCUS_ERR_INVALID_ARG;
  if (n_sink > 0 && !sink_idx) return FOCUS_ERR_INVALID_ARG;
  if (head_reduce != FOCUS_HEADS_PER_KV_GROUP && head_reduce != FOCUS_HEADS_ALL) return FOCUS_ERR_INVALID_ARG;
  if (sink_mode != FOCUS_SINK_TOKENS && sink_mode != FOCUS_SINK_BLOCKS) return FOCUS_ERR_INVALID_ARG;
  if (sink_mode == FOCUS_SINK_TOKENS && n_sink > 0 && !sink_keep) return FOCUS_ERR_INVALID_ARG;
  if (sink_mode == FOCUS_SINK_BLOCKS && max_blocks < (nb < C + n_sink ? nb : C + n_sink)) return FOCUS_ERR_INVALID_ARG;
  if (nb > SB_MAX_NB) return FOCUS_ERR_UNSUPPORTED;
  if (nb == 0 && max_blocks == 0) {
    // nothing to select; counts still have to be defined
  }
  const int G = head_reduce == FOCUS_HEADS_ALL ? 1 : shape->n_kv_heads;
  select_blocks_kernel<<<G, SB_THREADS, 0, stream>>>(R, nb, C, shape->kv_block, sink_idx, n_sink,
                                                     sink_mode == FOCUS_SINK_BLOCKS, block_idx, max_blocks, block_cnt,
                                                     sink_keep, ctx->d_status);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}

// ------------------------------------------------------------------------------------------------
// Stage 2, selection half.  sink_reduce_heads: S[j] = inv * sum_h part[h][j] in fixed head order.
// sink_topn: one CTA, 8-bit radix select of the n-th largest key, then ascending ordered compaction.
// ------------------------------------------------------------------------------------------------
__global__ void sink_reduce_heads_kernel(const float* __restrict__ part, int H, int L, const int32_t* n_active,
                                         float* __restrict__ S) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= L) return;
  float acc = 0.f;
  for (int h = 0; h < H; ++h) acc += part[(size_t)h * L + j];
  const int n = *n_active;
  S[j] = n > 0 ? acc / ((float)H * (float)n) : 0.f;
}

constexpr int TN_THREADS = 1024;
constexpr int TN_MAX_SMEM_KEYS = 50 * 1024;      // keys cached in shared memory (200 KB); beyond that they are re-read

// One CTA.  Keys (order-preserving integers of the scores) are staged once in shared memory, then:
// (1) the key T of the want-th largest element is found bit by bit, MSB first (T keeps a bit iff at least `want`
//     keys are >= the candidate): counting sweeps with no atomics per element.  Sink scores are all close to 1/L,
//     so (a) the bits on which all keys agree are found first (one AND/OR sweep) and skipped, and (b) as soon as
//     at most LIST_MAX keys are still undecided (same prefix as T) they are copied to a short list and the
//     remaining bits only look at the list;
// (2) the selected positions are written ascending.  If every key equal to T is taken (no tie is cut) they are
//     collected in any order and ranked by position; otherwise warp w walks the w-th contiguous segment of the
//     candidates (ballot/popc keeps index order, one block scan orders the warps) and keys equal to T are taken in
//     index order until the quota is filled.
constexpr int LIST_MAX = TN_THREADS;
constexpr int SEL_MAX = 4096;

template <bool CACHED>
__global__ void __launch_bounds__(TN_THREADS)
sink_topn_kernel(const float* __restrict__ S, int lo, int hi, int n_sink, const int32_t* n_active,
                 int32_t* __restrict__ sink_idx, int32_t* status) {
  extern __shared__ uint32_t skey[];
  __shared__ int cnt[40];
  __shared__ int scan_s[33];
  __shared__ uint32_t s_and, s_or;
  __shared__ uint32_t list[LIST_MAX];
  __shared__ int sel[SEL_MAX];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = hi - lo;
  const int want = min(n_sink, n);
  if (n_active && *n_active <= 0) {          // undefined scores: report and emit an empty set (NULL: scores as given)
    if (tid == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
    for (int i = tid; i < n_sink; i += TN_THREADS) sink_idx[i] = -1;
    publish_outputs();
    return;
  }
  if (want == 0) {
    for (int i = tid; i < n_sink; i += TN_THREADS) sink_idx[i] = -1;
    publish_outputs();
    return;
  }
  if (tid < 40) cnt[tid] = 0;
  if (tid == 0) { s_and = 0xFFFFFFFFu; s_or = 0u; }
  if (CACHED) {
#pragma unroll 8
    for (int i = tid; i < n; i += TN_THREADS) skey[i] = float_key(S[lo + i]);
  }
  __syncthreads();
  auto key_at = [&](int i) -> uint32_t { return CACHED ? skey[i] : float_key(S[lo + i]); };
  auto count_ge = [&](uint32_t cand, int slot) -> int {          // block-wide count of keys >= cand (one barrier)
    int c = 0;
#pragma unroll 8
    for (int i = tid; i < n; i += TN_THREADS) c += key_at(i) >= cand ? 1 : 0;
    c = __reduce_add_sync(0xffffffffu, c);
    if (lane == 0 && c) atomicAdd(&cnt[slot], c);
    __syncthreads();
    return cnt[slot];
  };
  // bits shared by all keys
  {
    uint32_t a = 0xFFFFFFFFu, o = 0u;
#pragma unroll 8
    for (int i = tid; i < n; i += TN_THREADS) { const uint32_t k = key_at(i); a &= k; o |= k; }
    a = __reduce_and_sync(0xffffffffu, a);
    o = __reduce_or_sync(0xffffffffu, o);
    if (lane == 0) { atomicAnd(&s_and, a); atomicOr(&s_or, o); }
    __syncthreads();
  }
  const uint32_t diff = s_and ^ s_or;
  const int hb = diff ? 31 - __clz(diff) : -1;                    // highest bit on which two keys differ
  uint32_t T = hb >= 0 ? (s_or & ~((2u << hb) - 1u)) : s_or;      // common prefix, lower bits still open
  if (hb == 31) T = 0u;
  int lo_cnt = n, hi_cnt = 0;                                     // keys >= T; keys >= T + 2^(bit+1)
  int bit = hb;
  for (; bit >= 0 && lo_cnt - hi_cnt > LIST_MAX; --bit) {
    const uint32_t cand = T | (1u << bit);
    const int c = count_ge(cand, bit);
    if (c >= want) { T = cand; lo_cnt = c; } else { hi_cnt = c; }
  }
  if (bit >= 0) {
    // undecided keys (prefix above `bit` equal to T's) -> list; the remaining bits only look at the list
    const uint32_t top = bit == 31 ? 0u : (T >> (bit + 1));
#pragma unroll 4
    for (int i = tid; i < n; i += TN_THREADS) {
      const uint32_t k = key_at(i);
      if ((bit == 31 ? 0u : (k >> (bit + 1))) == top) list[atomicAdd(&cnt[32], 1)] = k;
    }
    __syncthreads();
    const int nl = cnt[32];
    const uint32_t mine = tid < nl ? list[tid] : 0u;
    const int above = hi_cnt;                    // keys above the listed range: they are >= every further candidate
    for (; bit >= 0; --bit) {
      const uint32_t cand = T | (1u << bit);
      int c = (tid < nl && mine >= cand) ? 1 : 0;
      c = __reduce_add_sync(0xffffffffu, c);
      if (lane == 0 && c) atomicAdd(&cnt[bit], c);
      __syncthreads();
      const int tot = above + cnt[bit];
      if (tot >= want) { T = cand; lo_cnt = tot; } else { hi_cnt = tot; }
    }
  }
  // T = key of the want-th largest element; hi_cnt = keys > T; lo_cnt - hi_cnt = keys == T
  const int remaining = want - hi_cnt;           // how many keys == T to take (lowest index first)
  if (remaining == lo_cnt - hi_cnt && want <= SEL_MAX) {
    // no tie is cut: the selected set is {key >= T}; collect in any order, then rank by position
#pragma unroll 4
    for (int i = tid; i < n; i += TN_THREADS)
      if (key_at(i) >= T) sel[atomicAdd(&cnt[33], 1)] = lo + i;
    __syncthreads();
    for (int t = tid; t < want; t += TN_THREADS) {
      const int mine = sel[t];
      int rank = 0;
      for (int j = 0; j < want; ++j) rank += sel[j] < mine ? 1 : 0;
      sink_idx[rank] = mine;
    }
    for (int i = want + tid; i < n_sink; i += TN_THREADS) sink_idx[i] = -1;
    publish_outputs();
    return;
  }
  // ordered compaction: warp w owns candidates [w*seg, (w+1)*seg), seg a multiple of 32
  const int seg = ((n + 31) / 32 + 31) / 32 * 32;
  const int w_lo = min(warp * seg, n), w_hi = min(w_lo + seg, n);
  int n_gt = 0, n_eq = 0;
  for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t k = i < w_hi ? key_at(i) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, i < w_hi && k > T));
    n_eq += __popc(__ballot_sync(0xffffffffu, i < w_hi && k == T));
  }
  int tot_eq, tot_sel;
  const int pre_eq = block_excl_scan(lane == 0 ? n_eq : 0, scan_s, tot_eq);          // per-warp values on lane 0
  const int w_pre_eq = __shfl_sync(0xffffffffu, pre_eq, 0);
  const int take_eq = max(0, min(n_eq, remaining - w_pre_eq));                       // equals are taken in index order
  const int pre_sel = block_excl_scan(lane == 0 ? n_gt + take_eq : 0, scan_s, tot_sel);
  int out = __shfl_sync(0xffffffffu, pre_sel, 0), eq_seen = 0;
  for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t k = i < w_hi ? key_at(i) : 0u;
    const uint32_t m_eq = __ballot_sync(0xffffffffu, i < w_hi && k == T);
    const int my_eq_rank = eq_seen + __popc(m_eq & ((1u << lane) - 1u));
    const bool take = i < w_hi && (k > T || (k == T && my_eq_rank < take_eq));
    const uint32_t m_take = __ballot_sync(0xffffffffu, take);
    if (take) sink_idx[out + __popc(m_take & ((1u << lane) - 1u))] = lo + i;
    out += __popc(m_take);
    eq_seen += __popc(m_eq);
  }
  for (int i = tot_sel + tid; i < n_sink; i += TN_THREADS) sink_idx[i] = -1;
  publish_outputs();
}

// ------------------------------------------------------------------------------------------------
// Stage 2, selection half, on one thread-block cluster (SC_CTAS CTAs): exact Top-n of the head-reduced scores and
// the ascending index list.  CTA r owns the r-th contiguous chunk of the candidates, keeps their
// order-preserving keys in shared memory and never looks at another CTA's keys; what the CTAs exchange through
// distributed shared memory are a few words per step:
//   (1) AND / OR of all keys  -> the bits on which every key agrees are skipped (sink scores all sit near 1/L);
//   (2) per 8-bit digit, MSB first, a 256-bin histogram of the keys that still match the prefix of the n-th largest
//       key T: every CTA adds up the SC_CTAS histograms and takes the same decision (two histogram buffers in turn,
//       so one cluster barrier per digit suffices);
//   (3) per CTA the number of keys > T and == T: keys equal to T are taken in global index order until the quota
//       is filled, which fixes every CTA's output offset and its share of the equals.
// Inside a CTA the selected positions are written ascending by warp-ordered ballot compaction.
// ------------------------------------------------------------------------------------------------
constexpr int SC_CTAS = 8;
constexpr int SC_THREADS = 1024;
constexpr int SC_MAX_KEYS = 48 * 1024;                 // keys per CTA (192 KB of dynamic shared memory)

__device__ __forceinline__ uint32_t sc_map(const void* p, uint32_t rank) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p), r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
  return r;
}
__device__ __forceinline__ uint32_t sc_ld(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sc_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(SC_THREADS, 1)
sink_select_cluster_kernel(const float* __restrict__ S, const int32_t* n_active, int lo, int hi, int n_sink,
                           int32_t* __restrict__ sink_idx, int32_t* status) {
  extern __shared__ uint32_t skey[];                    // this CTA's keys
  __shared__ uint32_t xch[4];                           // and, or, #keys > T, #keys == T of this CTA
  __shared__ uint32_t hist[2][256];
  __shared__ uint32_t tot[256];
  __shared__ int scan_s[33];
  __shared__ int s_digit, s_above;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int n = hi - lo;
  const int want = min(n_sink, n);
  const int n_act = n_active ? *n_active : 1;           // NULL: the scores are taken as given
  const int chunk = (n + SC_CTAS - 1) / SC_CTAS;
  const int c_lo = min((int)rank * chunk, n), c_hi = min(c_lo + chunk, n), cn = c_hi - c_lo;
  uint32_t a = 0xFFFFFFFFu, o = 0u;
#pragma unroll 4
  for (int i = tid; i < cn; i += SC_THREADS) {
    const uint32_t k = float_key(S[lo + c_lo + i]);
    skey[i] = k;
    a &= k; o |= k;
  }
  if (n_act <= 0 || want == 0) {                        // undefined scores or nothing asked for: an empty set
    if (n_act <= 0 && tid == 0 && rank == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
    for (int i = (int)rank * SC_THREADS + tid; i < n_sink; i += SC_CTAS * SC_THREADS) sink_idx[i] = -1;
    publish_outputs();
    return;                                             // uniform over the cluster: nobody waits at a barrier
  }
  if (tid < 256) { hist[0][tid] = 0u; hist[1][tid] = 0u; }
  if (tid == 0) { xch[0] = 0xFFFFFFFFu; xch[1] = 0u; }
  __syncthreads();
  a = __reduce_and_sync(0xffffffffu, a);
  o = __reduce_or_sync(0xffffffffu, o);
  if (lane == 0) { atomicAnd(&xch[0], a); atomicOr(&xch[1], o); }
  __syncthreads();
  sc_sync();
  uint32_t g_and = 0xFFFFFFFFu, g_or = 0u;
#pragma unroll
  for (int r = 0; r < SC_CTAS; ++r) { g_and &= sc_ld(sc_map(&xch[0], r)); g_or |= sc_ld(sc_map(&xch[1], r)); }
  const uint32_t diff = g_and ^ g_or;
  int hb = diff ? 31 - __clz(diff) : -1;                // highest bit on which two keys differ
  // T: key of the want-th largest element, built digit by digit below the common prefix
  uint32_t T = hb >= 31 ? 0u : (hb >= 0 ? (g_or & ~((2u << hb) - 1u)) : g_or);
  int need = want;                                      // rank of T among the keys that share its prefix (1 = largest)
  int pass = 0;
  while (hb >= 0) {
    const int shift = hb >= 7 ? hb - 7 : 0;             // digit = bits [shift, shift + width)
    const int width = hb - shift + 1;
    const uint32_t dmask = (1u << width) - 1u;
    const uint32_t pmask = (hb >= 31) ? 0u : ~((2u << hb) - 1u);     // prefix bits above the digit
    uint32_t* hs = hist[pass & 1];
    for (int i = tid; i < cn; i += SC_THREADS) {
      const uint32_t k = skey[i];
      if ((k & pmask) == (T & pmask)) atomicAdd(&hs[(k >> shift) & dmask], 1u);
    }
    __syncthreads();
    sc_sync();
    if (tid < 256) {
      uint32_t t = 0u;
#pragma unroll
      for (int r = 0; r < SC_CTAS; ++r) t += sc_ld(sc_map(&hs[tid], r));
      tot[tid] = t;
      // the other buffer is cleared for the next digit: whoever read it (previous digit) did so before arriving at
      // the barrier above
      hist[(pass + 1) & 1][tid] = 0u;
    }
    __syncthreads();
    if (warp == 0) {
      // digits from the largest down: the first one whose cumulative count reaches `need`
      int run = 0, found = -1, above = 0;
      for (int base = 255; base >= 0 && found < 0; base -= 32) {
        const int d = base - lane;                      // lane 0 holds the largest digit of this group of 32
        const int c = (int)tot[d];
        int inc = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, inc, off);
          if (lane >= off) inc += y;
        }
        const uint32_t hit = __ballot_sync(0xffffffffu, run + inc >= need);
        if (hit) {
          const int l0 = __ffs(hit) - 1;
          found = base - l0;
          above = run + __shfl_sync(0xffffffffu, inc - c, l0);
        }
        run += __shfl_sync(0xffffffffu, inc, 31);
      }
      if (lane == 0) { s_digit = found; s_above = above; }
    }
    __syncthreads();
    const int d = s_digit;
    T |= (uint32_t)d << shift;
    need -= s_above;
    hb = shift - 1;
    ++pass;
    __syncthreads();
  }
  // keys > T and == T of this CTA
  int n_gt_l = 0, n_eq_l = 0;
  for (int i = tid; i < cn; i += SC_THREADS) {
    const uint32_t k = skey[i];
    n_gt_l += k > T ? 1 : 0;
    n_eq_l += k == T ? 1 : 0;
  }
  n_gt_l = __reduce_add_sync(0xffffffffu, n_gt_l);
  n_eq_l = __reduce_add_sync(0xffffffffu, n_eq_l);
  if (tid == 0) { xch[2] = 0u; xch[3] = 0u; }
  __syncthreads();
  if (lane == 0) { atomicAdd(&xch[2], (uint32_t)n_gt_l); atomicAdd(&xch[3], (uint32_t)n_eq_l); }
  __syncthreads();
  sc_sync();
  int gt_all = 0;
#pragma unroll
  for (int r = 0; r < SC_CTAS; ++r) gt_all += (int)sc_ld(sc_map(&xch[2], r));
  const int remaining = want - gt_all;                  // keys == T to take, lowest index first
  int out_base = 0, eq_before = 0, my_eq = 0;
#pragma unroll
  for (int r = 0; r < SC_CTAS; ++r) {
    const int g = (int)sc_ld(sc_map(&xch[2], r)), e = (int)sc_ld(sc_map(&xch[3], r));
    const int take = max(0, min(e, remaining - eq_before));
    if (r < (int)rank) out_base += g + take;
    if (r == (int)rank) my_eq = take;
    eq_before += e;
  }
  // ordered compaction inside the CTA: warp w owns keys [w*seg, (w+1)*seg), seg a multiple of 32
  const int seg = ((cn + 31) / 32 + 31) / 32 * 32;
  const int w_lo = min(warp * seg, cn), w_hi = min(w_lo + seg, cn);
  int n_gt = 0, n_eq = 0;
  for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t k = i < w_hi ? skey[i] : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, i < w_hi && k > T));
    n_eq += __popc(__ballot_sync(0xffffffffu, i < w_hi && k == T));
  }
  int tot_eq, tot_sel;
  const int pre_eq = block_excl_scan(lane == 0 ? n_eq : 0, scan_s, tot_eq);          // per-warp values on lane 0
  const int w_pre_eq = __shfl_sync(0xffffffffu, pre_eq, 0);
  const int take_eq = max(0, min(n_eq, my_eq - w_pre_eq));                           // equals are taken in index order
  const int pre_sel = block_excl_scan(lane == 0 ? n_gt + take_eq : 0, scan_s, tot_sel);
  int out = out_base + __shfl_sync(0xffffffffu, pre_sel, 0), eq_seen = 0;
  for (int i0 = w_lo; i0 < w_hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t k = i < w_hi ? skey[i] : 0u;
    const uint32_t m_eq = __ballot_sync(0xffffffffu, i < w_hi && k == T);
    const int my_eq_rank = eq_seen + __popc(m_eq & ((1u << lane) - 1u));
    const bool take = i < w_hi && (k > T || (k == T && my_eq_rank < take_eq));
    const uint32_t m_take = __ballot_sync(0xffffffffu, take);
    if (take) sink_idx[out + __popc(m_take & ((1u << lane) - 1u))] = lo + c_lo + i;
    out += __popc(m_take);
    eq_seen += __popc(m_eq);
  }
  for (int i = want + (int)rank * SC_THREADS + tid; i < n_sink; i += SC_CTAS * SC_THREADS) sink_idx[i] = -1;
  publish_outputs();
  sc_sync();                                            // nobody leaves while its shared memory may still be read
}

focus_status launch_sink_topn(focus_ctx* ctx, const float* S, const int32_t* n_active, int cand_lo, int cand_hi,
                              int n_sink, int32_t* sink_idx, cudaStream_t st);

focus_status launch_sink_select(focus_ctx* ctx, const float* part, int H, int L, const int32_t* n_active, float* S,
                                int cand_lo, int cand_hi, int n_sink, int32_t* sink_idx, cudaStream_t st) {
  sink_reduce_heads_kernel<<<(L + 255) / 256, 256, 0, st>>>(part, H, L, n_active, S);
  FOCUS_CHECK_LAUNCH();
  if (n_sink == 0) return FOCUS_OK;                     // scores only
  return launch_sink_topn(ctx, S, n_active, cand_lo, cand_hi, n_sink, sink_idx, st);
}

// Exact Top-n of given scores (n_active NULL: the scores are defined whatever produced them).
focus_status launch_sink_topn(focus_ctx* ctx, const float* S, const int32_t* n_active, int cand_lo, int cand_hi,
                              int n_sink, int32_t* sink_idx, cudaStream_t st) {
  const int n = cand_hi - cand_lo;
  const int chunk = (n + SC_CTAS - 1) / SC_CTAS;
  int& cluster_state = ctx->ls.select_cluster;        // 0 not tried, 1 works, 2 the cluster launch was refused once
  // the cluster pays for its barriers (about 1.5 us each, seven to eight of them) once a single CTA's sweeps over
  // all keys cost more: measured cross-over between 8K and 16K candidates
  if (n >= 12288 && chunk <= SC_MAX_KEYS && cluster_state != 2) {
    bool& attr_set = ctx->ls.select_attr_set;
    if (!attr_set) {
      if (cudaFuncSetAttribute(sink_select_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               SC_MAX_KEYS * 4) != cudaSuccess)
        return FOCUS_ERR_CUDA;
      attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(SC_CTAS, 1, 1); cfg.blockDim = dim3(SC_THREADS, 1, 1);
    cfg.dynamicSmemBytes = (size_t)chunk * 4; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = SC_CTAS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, sink_select_cluster_kernel, (const float*)S, n_active, cand_lo, cand_hi, n_sink, sink_idx,
                           ctx->d_status) == cudaSuccess) {
      cluster_state = 1;
      FOCUS_CHECK_LAUNCH();
      return FOCUS_OK;
    }
    cudaGetLastError();
    cluster_state = 2;                                // fall through to the one-CTA kernels
  }
  if (n <= TN_MAX_SMEM_KEYS) {
    bool& attr_set = ctx->ls.topn_attr_set;
    if (!attr_set) {
      if (cudaFuncSetAttribute(sink_topn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               TN_MAX_SMEM_KEYS * 4) != cudaSuccess)
        return FOCUS_ERR_CUDA;
      attr_set = true;
    }
    sink_topn_kernel<true><<<1, TN_THREADS, (size_t)n * 4, st>>>(S, cand_lo, cand_hi, n_sink, n_active, sink_idx,
                                                                ctx->d_status);
  } else {
    sink_topn_kernel<false><<<1, TN_THREADS, 0, st>>>(S, cand_lo, cand_hi, n_sink, n_active, sink_idx, ctx->d_status);
  }
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}
