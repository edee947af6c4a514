// Block-sparse / dense bidirectional attention on the 5th-generation tensor cores (Eq. 9; FullAttn of
// Algorithm 1).  bf16 inputs, head_dim 128 (or 64: the kernels keep their 128-wide geometry and leave the upper half
// of every operand tile out), fp32 accumulation in TMEM.
//
// attn_tc_kernel: one CTA = one 128-row query tile of one KV head (GQA: the rows of all query heads of the group
// are stacked, so every K/V tile is read once per group) x one contiguous range ("split") of that head's key
// tiles.  Key tiles are 128 keys wide and are enumerated from the selected block list (one 128-token block, or two
// 64-token blocks side by side, per tile), the gathered sink tokens and the response region; K/V tiles arrive by
// TMA through a ring of four slots, three of them in use when the key loop is short (see the launcher).
//
// Warp roles (192 threads):
//   warp 0        TMA producer (one lane): K0, K1, V0, K2, V1, ... in the order the MMA warp consumes them
//   warp 1        tcgen05.mma issuer (one lane) + TMEM allocation: S_b = Q K_j^T (b = j mod 2), O += P_j V_j in two
//                 halves of 64 keys
//   warps 2..5    online softmax, one query row per thread: S_b -> registers, exp2 in chunks of 32 keys, bf16 P back
//                 into TMEM (aliasing S_b) and handed over half by half, lazy rescale of O, final normalisation
// The splits of a query tile form a thread-block cluster and merge their partials (unnormalised O, running max,
// running sum) through distributed shared memory in fixed split order; when the clusters of a launch would not all
// be resident, partials go through global memory instead (last-arriving CTA or a second kernel merges).  Results
// are deterministic either way.
//
// attn_tc_wide_kernel<false> (further down): two query tiles per CTA for the tensor-bound regime;
// attn_tc_wide_kernel<true>: one query tile, two softmax warpgroups on alternating key tiles, for query sets with at
// least one full tile of rows that the two-tile form does not take.
//
// Every launch is a programmatic dependent launch: see the comment on p.pdl in attn_tc_kernel.
#include <stdio.h>
#include <stdlib.h>

#include "tc_common.cuh"

using namespace tc;

namespace {

constexpr int TM = 128;            // query rows per CTA
constexpr int TN = 128;            // keys per tile
constexpr int HD = 128;            // head dim
constexpr int NSLOT = 4;           // K/V ring slots
constexpr int EARLY = 3;           // copies requested when a CTA starts (K0, K1, V0); the others follow once K0 has landed
constexpr int RING_SHORT = 3, RING_LONG = 4;   // ring slots in use: key loops of fewer than 12 tiles per CTA, longer ones
static_assert(EARLY <= RING_SHORT && RING_LONG <= NSLOT, "ring");
constexpr int SLOT_BYTES = TN * HD * 2;
constexpr int HALF_BYTES = SLOT_BYTES / 2;     // one 64-wide half of a tile: 128 rows x 128 bytes
constexpr int Q_BYTES = TM * HD * 2;
constexpr int NBAR = 2 * NSLOT + 8;
constexpr int MAXT = 128;            // key tiles of a split whose descriptors are staged in shared memory
constexpr int SMEM_BYTES = 1024 + Q_BYTES + NSLOT * SLOT_BYTES + NBAR * 8 + 64 + MAXT * 8;
constexpr int NTHREADS = 192;
constexpr int PREF_TILES = 1;                  // key tiles (K and V) warmed in L2 ahead of the dependency wait
constexpr float RESCALE_THRESHOLD = 8.0f;      // log2 units: O is rescaled only when the row max grew by more
// which kernel form a launch takes (measured cross-overs, see the launcher)
constexpr int WIDE_MIN_TILES = 24;             // two-tile form: at least this many key tiles per CTA
constexpr int KP_MIN_ROWS = 128;               // key-pair form: at least this many stacked rows per KV head ...
constexpr int KP_MIN_TILES = 4;                // ... and this many key tiles per CTA

struct TcParams {
  const __nv_bfloat16* Q;
  __nv_bfloat16* O;
  float* lse;
  const int32_t* q_rows;
  const int32_t* n_rows;
  const int32_t* block_idx;
  const int32_t* block_cnt;
  const uint8_t* sink_mask;    // [Hkv][ns_pad]: 1 = attend this gathered sink column
  float* part_O;               // [cta][128][128] unnormalised partial outputs (n_splits > 1)
  float* part_ml;              // [cta][128][2] running max (log2 domain) and running sum
  int32_t* counters;           // one arrival counter per (KV head, query tile); NULL: a separate kernel merges the splits
  long long q_stride_row, q_stride_head;
  int q_base, n_q, rows_bound, L, M, H, Hkv, hpg, B, nb, dense, group_stride, max_blocks, n_sink, ns_pad;
  int n_mtiles, n_splits, lse_stride;
  int cluster;                 // 1: the splits of a tile are one thread-block cluster and merge through shared memory
  int pdl;                     // 1: launched as a programmatic dependent of the selection kernel (see the wait below)
  int ring;                    // one-tile kernel: K/V ring slots in use (EARLY <= ring <= NSLOT)
  int hd;                      // head dim: 128, or 64 (the upper 64 columns of every operand tile are then zeros)
  int pair;                    // 1: 64-token KV blocks, two selected blocks per 128-key tile; tmK / tmV have 64-row boxes
  float scale_log2;            // softmax scale * log2(e)
  int32_t* status;
};


struct TileInfo {
  int kind;     // 0: tile of the K/V tensors, 1: tile of the gathered sink rows
  int start;    // first key row of the tile in its tensor
  int nvalid;   // leading columns that are real keys (the rest is masked out)
  int start2;   // pair mode, kind 0: first key row of the tile's second half (columns 64..127)
};
// staged form of a TileInfo: x = start | kind << 30; y = nvalid | code << 8, code = start2 / 64 for a pair of
// blocks, all ones for "the 64 rows after the first half"
constexpr int START2_NEXT = 0x7FFFFF;
__device__ __forceinline__ int2 pack_tile(const TileInfo& ti) {
  const int code = ti.start2 == ti.start + 64 ? START2_NEXT : (ti.start2 >> 6);
  return make_int2(ti.start | (ti.kind << 30), ti.nvalid | (code << 8));
}
__device__ __forceinline__ TileInfo unpack_tile(int2 e) {
  TileInfo ti;
  ti.kind = e.x >> 30; ti.start = e.x & 0x3FFFFFFF; ti.nvalid = e.y & 0xff;
  const int code = (e.y >> 8) & START2_NEXT;
  ti.start2 = code == START2_NEXT ? ti.start + 64 : code << 6;
  return ti;
}

struct TileEnum {
  int n_blk;        // tiles that come from the block list (pair mode: two blocks per tile)
  int n_blocks;     // entries of the block list
  int n_sinkt, n_resp, total;
  const int32_t* blocks;
};

// The kernel parameters sit in constant memory that is new for every launch: the first touch of each line is a
// round trip to L2 or DRAM, and the code after the dependency wait walks through them one by one (measured: 1.8 us of
// the 3.1 us between the wait and the first TMA issue).  Touching one word per 32 bytes -- and the tensor maps --
// while the predecessor is still draining takes those misses off the critical path.
__device__ __forceinline__ void warm_params(const TcParams& p, const CUtensorMap* a, const CUtensorMap* b,
                                            const CUtensorMap* c, const CUtensorMap* d) {
  const unsigned w = (unsigned)(size_t)p.Q ^ (unsigned)(size_t)p.n_rows ^ (unsigned)(size_t)p.part_O ^
                     (unsigned)p.q_stride_head ^ (unsigned)p.Hkv ^ (unsigned)p.ns_pad ^ (unsigned)(size_t)p.status;
  asm volatile("" ::"r"(w));
  if (threadIdx.x == 0) {
    prefetch_tmap(a); prefetch_tmap(b);
    if (!p.dense) { prefetch_tmap(c); prefetch_tmap(d); }
  }
}

// First key tile of split s of n: floor(total * s / n).  total < 2^23 tiles (2^30 tokens) and s <= 8, so the product
// fits 32 bits (a 64-bit division is a subroutine of a few hundred cycles on the set-up path of every CTA).
__device__ __forceinline__ int split_lo(int total, int s, int n) {
  return (int)((unsigned)total * (unsigned)s / (unsigned)n);
}

__device__ __forceinline__ TileEnum make_enum(const TcParams& p, int g, int cnt_raw) {
  TileEnum e;
  if (p.dense) {
    e.n_blk = 0; e.n_blocks = 0; e.n_sinkt = 0; e.n_resp = (p.L + TN - 1) / TN; e.blocks = nullptr;
  } else {
    const int row = g * p.group_stride;
    e.n_blocks = min(max(cnt_raw, 0), p.max_blocks);
    e.n_blk = p.pair ? (e.n_blocks + 1) >> 1 : e.n_blocks;
    e.n_sinkt = p.ns_pad / TN;
    e.n_resp = (p.L - p.M + TN - 1) / TN;
    e.blocks = p.block_idx + (size_t)row * p.max_blocks;
  }
  e.total = e.n_blk + e.n_sinkt + e.n_resp;
  return e;
}

// First key tile of split s of n for a sparse key set, tiles weighed by what their softmax costs: a sink tile (one
// mask test per column) counts 3, a block or response tile 2.  With equal tile counts the split that got the sink
// tiles finished last and its cluster waited for it (config 2, four splits of 22 tiles: loops of 11.4 / 13.6 / 12.7 /
// 16.4 thousand cycles).  s = 0 gives 0, s = n the tile count; monotonic in s.
__device__ __forceinline__ int split_lo_cost(const TileEnum& e, int s, int n) {
  const unsigned wb = 2u * (unsigned)e.n_blk, ws = 3u * (unsigned)e.n_sinkt, W = wb + ws + 2u * (unsigned)e.n_resp;
  const unsigned x = (W * (unsigned)s + (unsigned)n - 1u) / (unsigned)n;          // ceil(W s / n)
  if (x <= wb) return (int)((x + 1u) / 2u);
  if (x <= wb + ws) return e.n_blk + (int)((x - wb + 2u) / 3u);
  return e.n_blk + e.n_sinkt + (int)((x - wb - ws + 1u) / 2u);
}

__device__ __forceinline__ TileInfo tile_info(const TcParams& p, const TileEnum& e, int t) {
  TileInfo ti;
  ti.start2 = -1;
  if (p.dense) {
    ti.kind = 0; ti.start = t * TN; ti.nvalid = min(TN, p.L - ti.start);
  } else if (t < e.n_blk && p.pair) {
    // two 64-token blocks side by side; a short block (the last one of the prompt) goes second so that the valid
    // columns stay a prefix; a missing second block repeats the first (finite data, masked out)
    int b0 = e.blocks[2 * t];
    int b1 = 2 * t + 1 < e.n_blocks ? e.blocks[2 * t + 1] : -2;
    ti.kind = 0;
    if (b0 < 0 || b0 >= p.nb || b1 == -1 || b1 < -2 || b1 >= p.nb) {  // reported once by the producer; fully masked
      ti.start = 0; ti.start2 = 0; ti.nvalid = 0;
    } else {
      if (b1 >= 0 && p.M - b0 * 64 < 64) { const int x = b0; b0 = b1; b1 = x; }
      ti.start = b0 * 64;
      const int n0 = min(64, p.M - ti.start);
      if (b1 >= 0) { ti.start2 = b1 * 64; ti.nvalid = n0 < 64 ? n0 : 64 + min(64, p.M - ti.start2); }
      else { ti.start2 = ti.start; ti.nvalid = n0; }
    }
  } else if (t < e.n_blk) {
    const int b = e.blocks[t];
    ti.kind = 0;
    if (b < 0 || b >= p.nb) {               // reported once by the producer; the tile is fully masked
      ti.start = 0; ti.nvalid = 0;
    } else {
      ti.start = b * p.B; ti.nvalid = min(p.B, p.M - ti.start);
    }
  } else if (t < e.n_blk + e.n_sinkt) {
    const int s = t - e.n_blk;
    ti.kind = 1; ti.start = s * TN; ti.nvalid = min(TN, p.n_sink - s * TN);
  } else {
    const int r = t - e.n_blk - e.n_sinkt;
    ti.kind = 0; ti.start = p.M + r * TN; ti.nvalid = min(TN, p.L - ti.start);
  }
  if (ti.start2 < 0) ti.start2 = ti.start + 64;
  return ti;
}

// One K or V tile into a ring slot (two 64-column halves, 128-byte swizzle).  Pair mode, tiles of the K/V tensors:
// the maps have 64-row boxes and each half of the key range comes from its own place (rows 64..127 of a half sit
// 8 KB, a whole number of swizzle atoms, after rows 0..63).
__device__ __forceinline__ void load_tile(const TcParams& p, const TileInfo& ti, const CUtensorMap* map, uint32_t dst,
                                          uint32_t bar, int g, uint64_t l2_pol) {
  const bool two = p.hd > 64;                     // head dim 64: only the lower half of the slot is filled (and read)
  mbar_expect_tx(bar, two ? SLOT_BYTES : HALF_BYTES);
  if (p.pair && ti.kind == 0) {
    tma_load_3d_hint(dst, map, bar, 0, ti.start, g, l2_pol);
    tma_load_3d_hint(dst + HALF_BYTES / 2, map, bar, 0, ti.start2, g, l2_pol);
    if (two) {
      tma_load_3d_hint(dst + HALF_BYTES, map, bar, 64, ti.start, g, l2_pol);
      tma_load_3d_hint(dst + HALF_BYTES + HALF_BYTES / 2, map, bar, 64, ti.start2, g, l2_pol);
    }
  } else {
    tma_load_3d_hint(dst, map, bar, 0, ti.start, g, l2_pol);
    if (two) tma_load_3d_hint(dst + HALF_BYTES, map, bar, 64, ti.start, g, l2_pol);
  }
}

// Merge of the split partials of one (KV head, query tile): out = sum_s 2^(m_s - m) O_s / sum_s 2^(m_s - m) l_s,
// splits taken in index order (deterministic whoever runs it).  Every step is an L2 round trip, so the work is
// laid out as two flat phases with many independent loads in flight: (1) one thread per row turns the per-split
// (max, sum) pairs into weights in shared memory, (2) one thread per (row, 4 columns) accumulates the outputs.
__device__ __forceinline__ void merge_rows(const TcParams& p, int tile, int g, int mt, int total_fr, float* wts) {
  const int rows = min(TM, total_fr - mt * TM);
  const int S = p.n_splits;
  float* inv_s = wts + TM * S;
  for (int row = threadIdx.x; row < rows; row += NTHREADS) {
    const float2* ml = reinterpret_cast<const float2*>(p.part_ml) + (size_t)tile * S * TM + row;
    float m = -INFINITY;
#pragma unroll 4
    for (int s = 0; s < S; ++s) {
      const float2 v = __ldcg(ml + (size_t)s * TM);
      if (v.y > 0.f) m = fmaxf(m, v.x);
    }
    float tot = 0.f;
#pragma unroll 4
    for (int s = 0; s < S; ++s) {
      const float2 v = __ldcg(ml + (size_t)s * TM);
      const float wgt = v.y > 0.f ? exp2f(v.x - m) : 0.f;
      tot += wgt * v.y;
      wts[row * S + s] = wgt;
    }
    inv_s[row] = tot > 0.f ? 1.f / tot : 0.f;
    if (p.lse) {
      const int fr = mt * TM + row;
      p.lse[(size_t)(g * p.hpg + fr % p.hpg) * p.lse_stride + fr / p.hpg] = (m + log2f(tot)) * 0.6931471805599453f;
    }
  }
  __syncthreads();
#pragma unroll 2
  for (int item = threadIdx.x; item < rows * 32; item += NTHREADS) {
    const int row = item >> 5, cg = item & 31;
    if (cg * 4 >= p.hd) continue;
    const float4* po = reinterpret_cast<const float4*>(p.part_O) + ((size_t)tile * S * TM + row) * (HD / 4) + cg;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int s = 0; s < S; ++s) {
      const float wgt = wts[row * S + s];
      const float4 o = __ldcg(po + (size_t)s * TM * (HD / 4));
      if (wgt > 0.f) { acc.x += wgt * o.x; acc.y += wgt * o.y; acc.z += wgt * o.z; acc.w += wgt * o.w; }
    }
    const float inv = inv_s[row];
    const int fr = mt * TM + row;
    __nv_bfloat16* orow = p.O + ((size_t)(fr / p.hpg) * p.H + (size_t)(g * p.hpg + fr % p.hpg)) * p.hd + cg * 4;
    uint2 v;
    v.x = pack_bf16(acc.x * inv, acc.y * inv);
    v.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(orow) = v;
  }
}

// ---- split merge inside a thread-block cluster ---------------------------------------------------------------
// When the n_splits CTAs of one (KV head, query tile) are launched as a cluster, each leaves its unnormalised
// partial (rows x 128 floats, row pitch PROW, plus (max, sum) per row) in its own shared memory; after a cluster
// barrier CTA `rank` merges the rows r with r mod n_splits == rank, reading every CTA's copy through distributed
// shared memory, splits in index order.  No global scratch, no fence, no atomic.
constexpr int PROW = HD + 4;                                   // floats per partial row (padding spreads the banks)

__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Exit barrier of a cluster: it only keeps every CTA (and its shared memory) alive until all peers have finished
// reading it, so it orders nothing -- relaxed arrive, plain wait.  A CTA arrives after the stores that consumed what
// it read from its peers, so none of its reads can still be in flight.  With release/acquire semantics the barrier
// also waited for those output stores to become visible (1.9 us after the last arrival against 0.8 us for the first
// barrier of the merge).
__device__ __forceinline__ void cluster_sync_exit() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_smem_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 ld_smem_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 ld_dsmem_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

// In-cluster merge for split counts up to SMAX.  One work item = one row x the 4-column groups c8, c8 + 8, c8 + 16,
// c8 + 24 (c8 = 0..7): the per-row work (weights, normaliser, addressing) is paid once per 16 output columns, and a
// quarter-warp reads 128 contiguous bytes of a partial.  The CTA's own partial is read with plain shared-memory
// loads, the others through the cluster window.
template <int ROWS, int NTH, int SMAX>
__device__ __forceinline__ void cluster_merge_items(const TcParams& p, int g, int mt, int rank, uint32_t spart, int mine, int tid) {
  constexpr int PART_ML_OFF = ROWS * PROW;                     // float offset of the (max, sum) pairs
  constexpr int KB = SMAX <= 4 ? 4 : 2;                        // column groups in flight per batch (register budget)
  const int S = p.n_splits;
  const int n_items = mine * 8;
  for (int item = tid; item < n_items; item += NTH) {
    const int row = rank + (item >> 3) * S, c8 = item & 7;
    float2 ml[SMAX];
#pragma unroll
    for (int s = 0; s < SMAX; ++s) {
      ml[s] = make_float2(0.f, 0.f);
      if (s < S) {
        const uint32_t off = (uint32_t)(PART_ML_OFF + row * 2) * 4u;
        ml[s] = s == rank ? ld_smem_f2(spart + off) : ld_dsmem_f2(map_to_rank(spart, (uint32_t)s) + off);
      }
    }
    float m = -INFINITY;
#pragma unroll
    for (int s = 0; s < SMAX; ++s)
      if (ml[s].y > 0.f) m = fmaxf(m, ml[s].x);
    float wgt[SMAX];
    float tot = 0.f;
#pragma unroll
    for (int s = 0; s < SMAX; ++s) {
      wgt[s] = ml[s].y > 0.f ? exp2f(ml[s].x - m) : 0.f;
      tot += wgt[s] * ml[s].y;
    }
    const float inv = tot > 0.f ? 1.f / tot : 0.f;
#pragma unroll
    for (int s = 0; s < SMAX; ++s) wgt[s] *= inv;
    const int fr = mt * ROWS + row;
    const int qr = fr / p.hpg, hh = fr % p.hpg;
    __nv_bfloat16* orow = p.O + ((size_t)qr * p.H + (size_t)(g * p.hpg + hh)) * p.hd;
#pragma unroll
    for (int k0 = 0; k0 < 4; k0 += KB) {
      float4 o[KB][SMAX];
#pragma unroll
      for (int k = 0; k < KB; ++k)
#pragma unroll
        for (int s = 0; s < SMAX; ++s)
          if (s < S) {
            const uint32_t off = (uint32_t)(row * PROW + (c8 + 8 * (k0 + k)) * 4) * 4u;
            o[k][s] = s == rank ? ld_smem_f4(spart + off) : ld_dsmem_f4(map_to_rank(spart, (uint32_t)s) + off);
          }
#pragma unroll
      for (int k = 0; k < KB; ++k) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < SMAX; ++s)
          if (s < S && wgt[s] > 0.f) {                           // an empty partial's accumulator is never read
            acc.x += wgt[s] * o[k][s].x; acc.y += wgt[s] * o[k][s].y;
            acc.z += wgt[s] * o[k][s].z; acc.w += wgt[s] * o[k][s].w;
          }
        uint2 v;
        v.x = pack_bf16(acc.x, acc.y);
        v.y = pack_bf16(acc.z, acc.w);
        if ((k0 + k) * 32 < p.hd) *reinterpret_cast<uint2*>(orow + (c8 + 8 * (k0 + k)) * 4) = v;
      }
    }
    if (p.lse && c8 == 0)
      p.lse[(size_t)(g * p.hpg + hh) * p.lse_stride + qr] = (m + log2f(tot)) * 0.6931471805599453f;
  }
}

// All threads of all CTAs of the cluster call this; the threads with 0 <= tid < NTH share the merge work.
template <int ROWS, int NTH>
__device__ __forceinline__ void cluster_merge(const TcParams& p, int g, int mt, int total_fr, int rank, uint32_t spart, int tid) {
  asm volatile("bar.sync 0;" ::: "memory");
  cluster_sync_all();
  const int rows = min(ROWS, total_fr - mt * ROWS);
  const int S = p.n_splits;                                   // <= 8 in cluster mode
  const int mine = rank < rows ? (rows - rank + S - 1) / S : 0;
  if (tid >= 0) {
    if (S <= 2) cluster_merge_items<ROWS, NTH, 2>(p, g, mt, rank, spart, mine, tid);
    else if (S <= 4) cluster_merge_items<ROWS, NTH, 4>(p, g, mt, rank, spart, mine, tid);
    else cluster_merge_items<ROWS, NTH, 8>(p, g, mt, rank, spart, mine, tid);
  }
  cluster_sync_exit();                                         // nobody leaves while its partial may still be read
}

// Called by every thread of every split CTA once its partial is written: the CTA that arrives last at the
// tile's counter merges all splits and re-arms the counter for the next launch.
__device__ __forceinline__ void finish_split(const TcParams& p, int tile, int g, int mt, int total_fr, int* s_last,
                                             float* wts) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(&p.counters[tile], 1);
    *s_last = prev == p.n_splits - 1;
    if (*s_last) p.counters[tile] = 0;
    __threadfence();
  }
  __syncthreads();
  if (*s_last) merge_rows(p, tile, g, mt, total_fr, wts);
}

__global__ void __launch_bounds__(NTHREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const __grid_constant__ CUtensorMap tmSK, const __grid_constant__ CUtensorMap tmSV, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.x / p.n_mtiles, mt = blockIdx.x % p.n_mtiles, split = blockIdx.y;
  const int W = p.ring;                              // ring slots in use (EARLY <= W <= NSLOT)

  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sptr = smem_raw + (sbase - smem_u32(smem_raw));
  const uint32_t sQ = sbase;
  const uint32_t sSlot = sbase + Q_BYTES;
  const uint32_t sBar = sSlot + NSLOT * SLOT_BYTES;
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (NSLOT + s); };
  auto bar_sfull = [&](int b) { return sBar + 8u * (2 * NSLOT + b); };
  auto bar_pready = [&](int b) { return sBar + 8u * (2 * NSLOT + 2 + b); };
  // P V of key tile idx commits to bar_pvdone(idx & 1): a softmax thread that has seen S of tile idx knows P V of
  // tile idx - 2 (and so idx - 3) complete, i.e. it is at most one phase behind on either barrier and a parity wait
  // cannot mistake a phase two further on for the one it asks for (with a single barrier it could: had the last
  // product retired before a delayed thread's first test, the test read "not yet" until the wait ran out)
  auto bar_pvdone = [&](int b) { return sBar + 8u * (b ? 2 * NSLOT + 7 : 2 * NSLOT + 4); };
  auto bar_pready2 = [&](int b) { return sBar + 8u * (2 * NSLOT + 5 + b); };   // second half (keys 64..127) of P_b stored
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(sptr + Q_BYTES + NSLOT * SLOT_BYTES + NBAR * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* s_last_p = reinterpret_cast<int*>(tmem_holder + 2);
  int2* tlist = reinterpret_cast<int2*>(tmem_holder + 16);      // (start | kind << 30, nvalid) per tile of this split

  // Programmatic dependent launch.  Every launch of this kernel lets its successor in the stream start early
  // (launch_dependents) and may itself have been started before its predecessor finished.  p.pdl = 2: the
  // predecessor is unknown, so nothing in global memory is touched before griddepcontrol.wait; only the private
  // set-up (barriers, TMEM) runs ahead.  p.pdl = 1: the predecessor is the selection kernel of the same sparse layer
  // (see further down).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (p.pdl) warm_params(p, &tmK, &tmV, &tmSK, &tmSV);
  auto arm_barriers = [&]() {                        // warp 0, lane 0
    for (int sl = 0; sl < NSLOT; ++sl) { mbar_init(bar_full(sl), 1); mbar_init(bar_empty(sl), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_sfull(b), 1); mbar_init(bar_pready(b), 128); mbar_init(bar_pready2(b), 128); }
    mbar_init(bar_pvdone(0), 1); mbar_init(bar_pvdone(1), 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  };
  auto alloc_tmem = [&]() {                          // warp 1, all lanes
    tmem_alloc(smem_u32(tmem_holder), 512);
    tmem_relinquish();
  };
  if (p.pdl == 2) {
    if (warp == 0 && lane == 0) arm_barriers();
    if (warp == 1) alloc_tmem();
    // While the predecessor drains (a CTA is resident a few microseconds before the wait returns), warm L2 with what
    // the chain of dependent loads after the wait will ask for: the row count and row list, this tile's query rows
    // and, for the dense key set (known without reading anything), the first K/V tiles.  Values read
    // here serve as prefetch addresses only (bounds-checked) and are read again after the wait.
    if (warp == 0 && lane == 0 && p.dense) {
      const int total = (p.L + TN - 1) / TN;
      const int pt0 = split_lo(total, split, p.n_splits), pt1 = split_lo(total, split + 1, p.n_splits);
      for (int t = pt0; t < pt1 && t < pt0 + PREF_TILES; ++t) {
        tma_prefetch_3d(&tmK, 0, t * TN, g); tma_prefetch_3d(&tmV, 0, t * TN, g);
        if (p.hd > 64) { tma_prefetch_3d(&tmK, 64, t * TN, g); tma_prefetch_3d(&tmV, 64, t * TN, g); }
      }
    }
    if (warp >= 2) {
      const int ptid = (int)threadIdx.x - 64;                            // 0..127: one query row each
      const int qr = (mt * TM + ptid) / p.hpg, hh = (mt * TM + ptid) % p.hpg;
      if (qr < p.rows_bound) {
        int pos = p.q_base + qr;
        if (p.q_rows) {
          if (ptid == 0) prefetch_l2(p.n_rows);
          pos = *reinterpret_cast<const volatile int*>(p.q_rows + qr);
        }
        if (pos >= p.q_base && pos < p.q_base + p.n_q) {
          const __nv_bfloat16* row = p.Q + (long long)(pos - p.q_base) * p.q_stride_row + (long long)(g * p.hpg + hh) * p.q_stride_head;
          prefetch_l2(row);
          if (p.hd > 64) prefetch_l2(row + 64);
        }
      }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
  }
  // Dense key set: which tiles this split streams is known without reading anything, so the first K/V copies
  // start right here, ahead of the chain row count -> row list -> query rows (about 3 us sooner than from their
  // usual place further down).  Should the tile then turn out to have no rows, the copies are awaited
  // before the CTA leaves.
  // the two loads every thread's set-up hangs on are requested first (their values are consumed further down)
  constexpr int QCH = HD * 2 / 16;                               // 16-byte chunks per query row
  const int qtid = (int)threadIdx.x - 64;                        // row of the tile staged by this thread (warps 2..5)
  const int nrows_raw = p.q_rows ? ld_ordered(p.n_rows) : p.n_q;
  const int my_fr = mt * TM + qtid;
  const int my_qr = my_fr / p.hpg, my_hh = my_fr - my_qr * p.hpg;
  const int my_pos = (qtid >= 0 && my_qr < p.rows_bound) ? (p.q_rows ? ld_ordered(p.q_rows + my_qr) : p.q_base + my_qr) : -1;
  int early_issued = 0;
  if (p.pdl == 2 && p.dense && warp == 0) {
    const int total = (p.L + TN - 1) / TN;
    const int pt0 = split_lo(total, split, p.n_splits), pt1 = split_lo(total, split + 1, p.n_splits);
    const int ntd = pt1 - pt0;
    const int n_e = 2 * ntd < EARLY ? 2 * ntd : EARLY;
    const uint64_t pol = l2_policy_evict_first();
    if (lane < n_e) {                                // lane q issues copy q: K0, K1, V0, K2, V1, ... as in seq_tile below
      const int q = lane;
      bool isV; int idx;
      if (q == 0) { isV = false; idx = 0; }
      else if (q == 2 * ntd - 1) { isV = true; idx = ntd - 1; }
      else if (q & 1) { isV = false; idx = (q + 1) >> 1; }
      else { isV = true; idx = (q >> 1) - 1; }
      TileInfo ti;
      ti.kind = 0; ti.start = (pt0 + idx) * TN; ti.nvalid = min(TN, p.L - ti.start); ti.start2 = ti.start + 64;
      load_tile(p, ti, isV ? &tmV : &tmK, sSlot + q * SLOT_BYTES, bar_full(q), g, pol);
    }
    early_issued = n_e;
    __syncwarp();
  }

  // The prologue is a chain of global-memory latencies; everything that does not depend on another load is
  // requested first: the row count and the position of this thread's query row.  Each of the 128 softmax threads
  // stages one whole row (sixteen 16-byte chunks): one row-list entry and one division per thread, and a short
  // stretch of straight-line code (the earlier chunk-interleaved mapping cost every thread sixteen of each).
  // The query row is requested as soon as its position is known, without waiting for the row count: an entry of
  // the row list beyond the count is either a valid position (a row read for nothing) or not (skipped).
  uint4 qv[QCH];
#pragma unroll
  for (int c = 0; c < QCH; ++c) qv[c] = make_uint4(0, 0, 0, 0);
  const bool pos_ok = my_pos >= p.q_base && my_pos < p.q_base + p.n_q;
  if (pos_ok) {
    const uint4* src = reinterpret_cast<const uint4*>(p.Q + (long long)(my_pos - p.q_base) * p.q_stride_row +
                                                      (long long)(g * p.hpg + my_hh) * p.q_stride_head);
#pragma unroll
    for (int c = 0; c < QCH; ++c)
      if (c * 8 < p.hd) qv[c] = ld_ordered(src + c);
  }
  const int nrows = p.q_rows ? min(max(nrows_raw, 0), p.rows_bound) : p.n_q;
  const int total_fr = nrows * p.hpg;                    // stacked (row, head-of-group) rows of this KV head
  if (mt * TM >= total_fr) {                             // uniform: nothing to compute for this tile
    if (p.pdl == 2) {                                    // TMEM was allocated ahead of the row count
      if (lane == 0)
        for (int q = 0; q < early_issued; ++q)           // copies already on their way land before the CTA leaves
          mbar_wait(bar_full(q), 0u, abort_flag, p.status);
      tc_fence_before();
      __syncthreads();
      tc_fence_after();
      if (warp == 1) {
        __syncwarp();
        tmem_dealloc(*tmem_holder, 512);
      }
    }
    return;
  }

  // a listed row whose position is out of range is reported; rows beyond the count are staged as zeros
  if (qtid >= 0 && my_fr < total_fr && !pos_ok) set_status(p.status, FOCUS_ERR_INVALID_ARG);
  if (my_fr >= total_fr) {
#pragma unroll
    for (int c = 0; c < QCH; ++c) qv[c] = make_uint4(0, 0, 0, 0);
  }
  auto store_q = [&]() {                             // softmax warps: row qtid, chunk c -> swizzled K-major tile
#pragma unroll
    for (int c = 0; c < QCH; ++c) {
      const int half = c >> 3, cc = c & 7;
      *reinterpret_cast<uint4*>(sptr + half * HALF_BYTES + qtid * 128 + ((cc ^ (qtid & 7)) << 4)) = qv[c];
    }
  };
  // Launched as a programmatic dependent of the selection kernel of the same sparse layer: everything above
  // (row list, query rows) does not come from that kernel and overlaps with it; the block lists, the gathered
  // sink rows and their mask do, so nothing below may start before it has completed.
  if (p.pdl == 1) {
    // as a programmatic dependent the whole private set-up runs while the selection kernel is still at work
    if (warp == 0 && lane == 0) arm_barriers();
    if (warp == 1) alloc_tmem();
    if (qtid >= 0) store_q();
    asm volatile("griddepcontrol.wait;" ::: "memory");
  }
  const int cnt_raw = p.dense ? 0 : ld_ordered(p.block_cnt + g * p.group_stride);

  const TileEnum te = make_enum(p, g, cnt_raw);
  const int t0 = p.dense ? split_lo(te.total, split, p.n_splits) : split_lo_cost(te, split, p.n_splits);
  const int t1 = p.dense ? split_lo(te.total, split + 1, p.n_splits) : split_lo_cost(te, split + 1, p.n_splits);
  const int nt = t1 - t0;
  const int cta_lin = blockIdx.x * p.n_splits + split;

  const bool use_list = !p.dense && nt <= MAXT;
  // tile descriptor: from the staged list (sparse) or by arithmetic (dense; splits longer than the list)
  auto get_tile = [&](int idx) -> TileInfo {
    if (use_list) {
      return unpack_tile(tlist[idx]);
    }
    return tile_info(p, te, t0 + idx);
  };

  if (nt <= 0 && p.pdl) {                                 // TMEM was allocated before the split turned out empty
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
      __syncwarp();
      tmem_dealloc(*tmem_holder, 512);
    }
  }
  if (nt <= 0 && p.cluster) {                             // empty split inside a cluster: neutral partial, then merge duty
    float* ps = reinterpret_cast<float*>(sptr + Q_BYTES);
    for (int r = threadIdx.x; r < TM; r += NTHREADS) { ps[TM * PROW + 2 * r] = -INFINITY; ps[TM * PROW + 2 * r + 1] = 0.f; }
    cluster_merge<TM, NTHREADS>(p, g, mt, total_fr, split, sSlot, (int)threadIdx.x);
    return;
  }
  if (nt <= 0) {                                          // empty split: publish a neutral partial
    if (p.n_splits > 1) {
      if (warp >= 2) {
        const int row = (warp & 3) * 32 + lane;
        if (mt * TM + row < total_fr) {
          p.part_ml[((size_t)cta_lin * TM + row) * 2 + 0] = -INFINITY;
          p.part_ml[((size_t)cta_lin * TM + row) * 2 + 1] = 0.f;
        }
      }
      if (p.counters) finish_split(p, blockIdx.x, g, mt, total_fr, s_last_p, reinterpret_cast<float*>(sptr + Q_BYTES));
    }
    return;
  }

  // ---- set-up -------------------------------------------------------------------------------------
  // Warp 0 arms the barriers, stages the tile list and requests the first copies (K0, K1, V0) right away: they
  // need nothing from the other warps, which meanwhile allocate TMEM and stage Q.
  // Load sequence q -> (tile, K or V), the order the MMA warp consumes: K0, K1, V0, K2, V1, ..., V(nt-1).
  auto seq_tile = [&](int q, bool& isV) -> int {
    if (q == 0) { isV = false; return 0; }
    if (q == 2 * nt - 1) { isV = true; return nt - 1; }
    if (q & 1) { isV = false; return (q + 1) >> 1; }
    isV = true; return (q >> 1) - 1;
  };
  const uint64_t l2_pol = l2_policy_evict_first();
  auto issue = [&](int q, int slot) {
    bool isV;
    const int idx = seq_tile(q, isV);
    const TileInfo ti = get_tile(idx);
    const CUtensorMap* map = ti.kind ? (isV ? &tmSV : &tmSK) : (isV ? &tmV : &tmK);
    load_tile(p, ti, map, sSlot + slot * SLOT_BYTES, bar_full(slot), g, l2_pol);
  };
  const int n_loads = 2 * nt;
  const int n_early = n_loads < EARLY ? n_loads : EARLY;
  if (warp == 0) {
    if (lane == 0 && !p.pdl) arm_barriers();
    if (use_list) {
      for (int t = lane; t < nt; t += 32) {
        const TileInfo ti = tile_info(p, te, t0 + t);
        if (t0 + t < te.n_blk && ti.nvalid == 0) set_status(p.status, FOCUS_ERR_INVALID_ARG);   // bad block index
        tlist[t] = pack_tile(ti);
      }
    }
    __syncwarp();
    if (lane >= early_issued && lane < n_early) issue(lane, lane);   // one copy per lane (EARLY <= W: slot = copy index)
    __syncwarp();
  }
  if (warp == 1 && !p.pdl) alloc_tmem();
  // Q tile -> shared memory in the 128-byte-swizzled K-major layout the MMA descriptor expects:
  // half h (columns 64h..64h+63) at h*16 KB, row r at r*128 bytes, 16-byte chunk c at ((c ^ (r & 7)) * 16).
  if (qtid >= 0 && p.pdl != 1) store_q();
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_holder;
  const uint32_t tmem_O = tmem + 256;

  if (warp == 0) {
    // ================================ TMA producer ================================================
    if (lane == 0) {
      int issued = n_early;
      bool ok = true;
      // All CTAs of a launch start together: with a whole ring requested at once the first key tile shares the
      // memory system with five others per CTA and lands when they all do.  The first score tile needs K0 only,
      // so the copies beyond the first three wait for it.
      if (n_early < n_loads) ok = mbar_wait(bar_full(0), 0u, abort_flag, p.status);
      int slot = n_early == W ? 0 : n_early;                 // slot and round of copy q, kept without dividing by W
      uint32_t round = n_early == W ? 1u : 0u;
      for (int q = n_early; q < n_loads && ok; ++q) {
        if (!mbar_wait(bar_empty(slot), (round & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
        issue(q, slot);
        ++issued;
        if (++slot == W) { slot = 0; ++round; }
      }
      if (!ok) {
        // unwinding: let the copies already issued land before the CTA's shared memory is released
        const uint32_t first = issued > W ? (uint32_t)(issued - W) : 0u;
        for (uint32_t i = first; i < (uint32_t)issued; ++i) {
          uint64_t t_start = global_ns();
          while (!mbar_try_wait(bar_full(i % W), (i / W) & 1u)) {
            if (global_ns() - t_start > WAIT_LIMIT_NS) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ==================================================
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = make_idesc(TM, TN, 0);
      const uint32_t IDESC_PV = p.hd > 64 ? make_idesc(TM, HD, 1) : make_idesc(TM, 64, 1);   // head dim 64: O is 64 columns wide
      const uint64_t qdesc = make_sdesc(sQ, 16, 1024);
      int slot = 0;                                          // ring slot and round of the next tile to consume
      uint32_t round = 0;
      bool ok = true;
      auto do_pv = [&](int idx) -> bool {
        const int b = idx & 1;
        if (!mbar_wait(bar_pready(b), (uint32_t)(idx >> 1) & 1u, abort_flag, p.status)) return false;
        if (!mbar_wait(bar_full(slot), round & 1u, abort_flag, p.status)) return false;
        tc_fence_after();
        const uint64_t vdesc = make_sdesc(sSlot + slot * SLOT_BYTES, HALF_BYTES, 1024);
        const uint32_t pt = tmem + b * 128;
#pragma unroll
        for (int ks = 0; ks < TN / 32; ++ks)
          mma_ts(tmem_O, pt + ks * 8, vdesc + (uint64_t)(ks * (2048 >> 4)), IDESC_PV, (idx > 0 || ks > 0) ? 1u : 0u);
        if (!mbar_wait(bar_pready2(b), (uint32_t)(idx >> 1) & 1u, abort_flag, p.status)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = TN / 32; ks < TN / 16; ++ks)
          mma_ts(tmem_O, pt + ks * 8, vdesc + (uint64_t)(ks * (2048 >> 4)), IDESC_PV, 1u);
        tc_commit(bar_empty(slot));
        tc_commit(bar_pvdone(b));
        if (++slot == W) { slot = 0; ++round; }
        return true;
      };
      for (int idx = 0; idx < nt && ok; ++idx) {
        const int b = idx & 1;
        if (!mbar_wait(bar_full(slot), round & 1u, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint64_t kdesc = make_sdesc(sSlot + slot * SLOT_BYTES, 16, 1024);
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            if (half == 1 && p.hd <= 64) continue;                   // head dim 64: one half of the contraction
            const uint64_t off = (uint64_t)((half * HALF_BYTES + ks * 32) >> 4);
            mma_ss(tmem + b * 128, qdesc + off, kdesc + off, IDESC_QK, (half | ks) ? 1u : 0u);
          }
        tc_commit(bar_empty(slot));
        tc_commit(bar_sfull(b));
        if (++slot == W) { slot = 0; ++round; }
        if (idx > 0) ok = do_pv(idx - 1);
      }
      if (ok) ok = do_pv(nt - 1);
    }
  } else {
    // ================================ softmax / epilogue ==========================================
    const int rq = warp & 3;                         // TMEM lane quarter this warp may access
    const int row = rq * 32 + lane;                  // query row of this thread inside the tile
    const uint32_t lane_off = (uint32_t)(rq * 32) << 16;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int idx = 0; idx < nt; ++idx) {
      const int b = idx & 1;
      // votes keep the warp together: the TMEM loads and stores below are warp-collective
      if (!__all_sync(0xffffffffu, mbar_wait(bar_sfull(b), (uint32_t)(idx >> 1) & 1u, abort_flag, p.status))) { ok = false; break; }
      tc_fence_after();
      uint32_t sreg[128];
      const uint32_t ts = tmem + lane_off + b * 128;
      TC_LD32(ts, (sreg + 0));
      TC_LD32(ts + 32, (sreg + 32));
      TC_LD32(ts + 64, (sreg + 64));
      TC_LD32(ts + 96, (sreg + 96));
      tc_wait_ld();
      const TileInfo ti = get_tile(idx);
      float tmax = -INFINITY;
      if (ti.kind == 0 && ti.nvalid == TN) {
        float t4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains instead of one of 128
#pragma unroll
        for (int c = 0; c < 128; c += 8) {
          t4[0] = fmax3(t4[0], __uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1]));
          t4[1] = fmax3(t4[1], __uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3]));
          t4[2] = fmax3(t4[2], __uint_as_float(sreg[c + 4]), __uint_as_float(sreg[c + 5]));
          t4[3] = fmax3(t4[3], __uint_as_float(sreg[c + 6]), __uint_as_float(sreg[c + 7]));
        }
        tmax = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
      } else if (ti.kind == 0) {
#pragma unroll
        for (int c = 0; c < 128; ++c) {
          const float v = c < ti.nvalid ? __uint_as_float(sreg[c]) : -INFINITY;
          sreg[c] = __float_as_uint(v);
          tmax = fmaxf(tmax, v);
        }
      } else {
        const uint32_t* mk = reinterpret_cast<const uint32_t*>(p.sink_mask + (size_t)g * p.ns_pad + ti.start);
#pragma unroll
        for (int c4 = 0; c4 < 32; ++c4) {
          const uint32_t mword = __ldg(mk + c4);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int c = c4 * 4 + e;
            const float v = ((mword >> (8 * e)) & 0xffu) ? __uint_as_float(sreg[c]) : -INFINITY;
            sreg[c] = __float_as_uint(v);
            tmax = fmaxf(tmax, v);
          }
        }
      }
      tmax *= p.scale_log2;                          // scale > 0: max commutes with the scaling
      float alpha = 1.f;
      bool rescale = false;
      if (tmax > m_ref + RESCALE_THRESHOLD) {        // also true for the first finite maximum (m_ref = -inf)
        if (m_ref != -INFINITY) {
          alpha = ex2(m_ref - tmax);
          rescale = true;
        }
        m_ref = tmax;
      }
      // p = 2^(s*scale_log2 - m_ref); a fully masked row so far (m_ref = -inf) contributes zeros
      const float mneg = m_ref == -INFINITY ? 0.f : -m_ref;
      if (idx > 0 && __any_sync(0xffffffffu, rescale)) {   // tcgen05.ld/st are warp-collective: the whole warp takes the branch
        // P_{idx-1} V_{idx-1} must have left the tensor core before O is touched (its barrier is at most one phase
        // behind: see bar_pvdone).
        if (!__all_sync(0xffffffffu, mbar_wait(bar_pvdone((idx - 1) & 1), (uint32_t)((idx - 1) >> 1) & 1u, abort_flag, p.status))) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t oreg[32];
          TC_LD32(tmem_O + lane_off + cb * 32, oreg);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) oreg[c] = __float_as_uint(__uint_as_float(oreg[c]) * alpha);
          TC_ST32(tmem_O + lane_off + cb * 32, oreg);
        }
      }
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {                 // 32 keys at a time: exponentials, bf16 P, row sum
        uint32_t preg[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int c = ch * 32 + 2 * i;
          float x0, x1;
          ffma2(x0, x1, __uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1]), p.scale_log2, p.scale_log2, mneg, mneg);
          const float p0 = ex2(x0), p1 = ex2(x1);
          preg[i] = pack_bf16(p0, p1);
          fadd2(acc[(i & 1) * 2], acc[(i & 1) * 2 + 1], acc[(i & 1) * 2], acc[(i & 1) * 2 + 1], p0, p1);
        }
        TC_ST16(ts + ch * 16, preg);
        if (ch == 1) {                                 // keys 0..63 of P are in place: the first half of P V may start
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(bar_pready(b));
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_pready2(b));
      l = l * alpha + ((acc[0] + acc[1]) + (acc[2] + acc[3]));
    }
    // ---- epilogue: wait for the last P V, normalise, write out -----------------------------------
    // The loop waits for a P V product only before a rescale: S_{nt-1} being complete says no more than that
    // P_{nt-3} V_{nt-3} is, which is the previous phase of the barrier of tile nt-1's parity.
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_pvdone((nt - 1) & 1), (uint32_t)((nt - 1) >> 1) & 1u, abort_flag, p.status));
    if (ok) {
      tc_fence_after();
      const int fr = mt * TM + row;
      const bool valid = fr < total_fr;
      if (p.n_splits == 1) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const int qr = valid ? fr / p.hpg : 0, hh = valid ? fr % p.hpg : 0;
        __nv_bfloat16* orow = p.O + ((size_t)qr * p.H + (size_t)(g * p.hpg + hh)) * p.hd;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t oreg[32];
          TC_LD32(tmem_O + lane_off + cb * 32, oreg);
          tc_wait_ld();
          if (valid) {
#pragma unroll
            for (int c = 0; c < 32; c += 8) {
              uint4 v;
              v.x = pack_bf16(__uint_as_float(oreg[c + 0]) * inv, __uint_as_float(oreg[c + 1]) * inv);
              v.y = pack_bf16(__uint_as_float(oreg[c + 2]) * inv, __uint_as_float(oreg[c + 3]) * inv);
              v.z = pack_bf16(__uint_as_float(oreg[c + 4]) * inv, __uint_as_float(oreg[c + 5]) * inv);
              v.w = pack_bf16(__uint_as_float(oreg[c + 6]) * inv, __uint_as_float(oreg[c + 7]) * inv);
              if (cb * 32 < p.hd) *reinterpret_cast<uint4*>(orow + cb * 32 + c) = v;
            }
          }
        }
        if (valid && p.lse)
          p.lse[(size_t)(g * p.hpg + hh) * p.lse_stride + qr] = (m_ref + log2f(l)) * 0.6931471805599453f;
      } else if (p.cluster) {
        if (__any_sync(0xffffffffu, valid)) {
          float* ps = reinterpret_cast<float*>(sptr + Q_BYTES);
          float* prow = ps + row * PROW;
#pragma unroll
          for (int cb = 0; cb < 4; ++cb) {
            uint32_t oreg[32];
            TC_LD32(tmem_O + lane_off + cb * 32, oreg);
            tc_wait_ld();
            if (valid) {
#pragma unroll
              for (int c = 0; c < 32; c += 4)
                *reinterpret_cast<uint4*>(prow + cb * 32 + c) = make_uint4(oreg[c], oreg[c + 1], oreg[c + 2], oreg[c + 3]);
            }
          }
          if (valid) { ps[TM * PROW + 2 * row] = m_ref; ps[TM * PROW + 2 * row + 1] = l; }
        }
      } else if (__any_sync(0xffffffffu, valid)) {           // warps whose 32 rows are all padding have nothing to publish
        float* po = p.part_O + ((size_t)cta_lin * TM + row) * HD;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t oreg[32];
          TC_LD32(tmem_O + lane_off + cb * 32, oreg);
          tc_wait_ld();
          if (valid) {
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              *reinterpret_cast<uint4*>(po + cb * 32 + c) = make_uint4(oreg[c], oreg[c + 1], oreg[c + 2], oreg[c + 3]);
          }
        }
        if (valid) {
          p.part_ml[((size_t)cta_lin * TM + row) * 2 + 0] = m_ref;
          p.part_ml[((size_t)cta_lin * TM + row) * 2 + 1] = l;
        }
      }
    }
  }
  // ---- teardown: every role converges here, also after a timed-out wait --------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, 512);
  }
  if (p.cluster) cluster_merge<TM, NTHREADS>(p, g, mt, total_fr, split, sSlot, (int)threadIdx.x);
  else if (p.n_splits > 1 && p.counters) finish_split(p, blockIdx.x, g, mt, total_fr, s_last_p, reinterpret_cast<float*>(sptr + Q_BYTES));
}

// ================================================================================================================
// Wide variant: one CTA = TWO 128-row query tiles (A, B) of one KV head.  Used when a KV head has at least 256
// stacked query rows (the gen-region query set), where the kernel is bound by the tensor pipe and by the
// exponentials rather than by HBM.  Every K/V tile is staged once and serves 256 rows; the two tiles take turns
// on the tensor core: while the softmax warps of A work on S_A(j), the tensor pipe runs S_B(j) = Q_B K_j^T and
// O_B += P_B(j-1) V_(j-1), and vice versa.  TMEM: S_A | S_B | O_A | O_B (4 x 128 columns), P aliases S.
// Warps (384 threads): 0 TMA producer, 1 MMA issuer + TMEM owner, 2..3 idle, 4..7 softmax of tile A, 8..11 softmax of
// tile B.  After set-up the first warpgroup hands most of its registers to the softmax warpgroups (setmaxnreg), which
// keep a whole 128-column score row per thread in registers.
// ================================================================================================================
constexpr int TMW = 256;
constexpr int NSLOT_W = 5;
constexpr int EARLY_W = 2;                      // copies requested when a CTA starts (K0, V0); the others follow once K0 has landed
constexpr int Q_BYTES_W = TMW * HD * 2;
constexpr int NBAR_W = 2 * NSLOT_W + 9;
constexpr int MAXT_W = 96;
constexpr int NTHREADS_W = 384;                 // three warpgroups: {producer, MMA, two idle warps}, softmax A, softmax B
constexpr int SMEM_BYTES_W = 1024 + Q_BYTES_W + NSLOT_W * SLOT_BYTES + NBAR_W * 8 + 64 + MAXT_W * 8;

// KP = false: the two softmax warpgroups own two different 128-row query tiles and share every key tile (above).
// KP = true ("key pair"): ONE 128-row query tile; warpgroup x takes the key tiles x, x + 2, x + 4, ... of the split
// with its own running maximum, row sum and accumulator (S_x, O_x), so that two softmax streams run per SM on a
// single query tile; the two halves are merged in the epilogue (each warpgroup reads both accumulators from TMEM
// for 64 of the 128 output columns).  Used when a KV head has too few rows or key tiles for the two-tile form.
template <bool KP>
__global__ void __launch_bounds__(NTHREADS_W, 1)
attn_tc_wide_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmSK, const __grid_constant__ CUtensorMap tmSV, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = blockIdx.x / p.n_mtiles, mt = blockIdx.x % p.n_mtiles, split = blockIdx.y;
  // programmatic dependent launch: let the successor start early; wait for the predecessor before touching memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (p.pdl) {
    warm_params(p, &tmK, &tmV, &tmSK, &tmSV);
    asm volatile("griddepcontrol.wait;" ::: "memory");
  }

  constexpr int TMQ = KP ? TM : TMW;                             // query rows of this CTA
  constexpr int QCH = HD * 2 / 16;                               // 16-byte chunks per query row
  // one query row per softmax thread (the key-pair form has 128 rows for 256 such threads: the upper half idles);
  // the row is requested as soon as its position is known, without waiting for the row count
  const int qtid = (int)threadIdx.x - 128;
  const bool stager = qtid >= 0 && qtid < TMQ;
  const int nrows_raw = p.q_rows ? ld_ordered(p.n_rows) : p.n_q;
  const int cnt_raw = p.dense ? 0 : ld_ordered(p.block_cnt + g * p.group_stride);
  const int my_fr = mt * TMQ + qtid;
  const int my_qr = my_fr / p.hpg, my_hh = my_fr - my_qr * p.hpg;
  const int my_pos = (stager && my_qr < p.rows_bound) ? (p.q_rows ? ld_ordered(p.q_rows + my_qr) : p.q_base + my_qr) : -1;
  uint4 qv[QCH];
#pragma unroll
  for (int c = 0; c < QCH; ++c) qv[c] = make_uint4(0, 0, 0, 0);
  const bool pos_ok = my_pos >= p.q_base && my_pos < p.q_base + p.n_q;
  if (pos_ok) {
    const uint4* src = reinterpret_cast<const uint4*>(p.Q + (long long)(my_pos - p.q_base) * p.q_stride_row +
                                                      (long long)(g * p.hpg + my_hh) * p.q_stride_head);
#pragma unroll
    for (int c = 0; c < QCH; ++c)
      if (c * 8 < p.hd) qv[c] = ld_ordered(src + c);
  }
  const int nrows = p.q_rows ? min(max(nrows_raw, 0), p.rows_bound) : p.n_q;
  const int total_fr = nrows * p.hpg;
  if (mt * TMQ >= total_fr) return;

  const TileEnum te = make_enum(p, g, cnt_raw);
  const int t0 = split_lo(te.total, split, p.n_splits);
  const int t1 = split_lo(te.total, split + 1, p.n_splits);
  const int nt = t1 - t0;

  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sptr = smem_raw + (sbase - smem_u32(smem_raw));
  const uint32_t sQ = sbase;
  const uint32_t sSlot = sbase + Q_BYTES_W;
  const uint32_t sBar = sSlot + NSLOT_W * SLOT_BYTES;
  auto bar_full = [&](int s) { return sBar + 8u * s; };
  auto bar_empty = [&](int s) { return sBar + 8u * (NSLOT_W + s); };
  auto bar_sfull = [&](int x) { return sBar + 8u * (2 * NSLOT_W + x); };
  auto bar_pready = [&](int x) { return sBar + 8u * (2 * NSLOT_W + 2 + x); };    // P_x columns of keys 0..63 stored
  auto bar_pready2 = [&](int x) { return sBar + 8u * (2 * NSLOT_W + 7 + x); };   // ... of keys 64..127
  auto bar_pvdone = [&](int x) { return sBar + 8u * (2 * NSLOT_W + 4 + x); };
  const uint32_t bar_alldone = sBar + 8u * (2 * NSLOT_W + 6);   // every MMA of this CTA has completed
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(sptr + Q_BYTES_W + NSLOT_W * SLOT_BYTES + NBAR_W * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int2* tlist = reinterpret_cast<int2*>(tmem_holder + 16);
  const bool use_list = !p.dense && nt <= MAXT_W;
  auto get_tile = [&](int idx) -> TileInfo {
    if (use_list) {
      return unpack_tile(tlist[idx]);
    }
    return tile_info(p, te, t0 + idx);
  };
  float* ps = reinterpret_cast<float*>(sptr + Q_BYTES_W);        // split partial (cluster mode), over the K/V ring

  if (nt <= 0) {                                                 // empty split (cluster mode only: see the launcher)
    for (int r = threadIdx.x; r < TMQ; r += NTHREADS_W) { ps[TMQ * PROW + 2 * r] = -INFINITY; ps[TMQ * PROW + 2 * r + 1] = 0.f; }
    cluster_merge<TMQ, 256>(p, g, mt, total_fr, split, sSlot, (int)threadIdx.x - 128);
    return;
  }

  // load sequence: q even -> K_(q/2), q odd -> V_(q/2); the MMA warp consumes K0, V0, K1, V1, ... in this order
  const uint64_t l2_pol = l2_policy_evict_first();
  auto issue = [&](int q) {
    const bool isV = q & 1;
    const TileInfo ti = get_tile(q >> 1);
    const int slot = q % NSLOT_W;
    const CUtensorMap* map = ti.kind ? (isV ? &tmSV : &tmSK) : (isV ? &tmV : &tmK);
    load_tile(p, ti, map, sSlot + slot * SLOT_BYTES, bar_full(slot), g, l2_pol);
  };
  const int n_loads = 2 * nt;
  const int n_early = n_loads < EARLY_W ? n_loads : EARLY_W;
  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < NSLOT_W; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
      for (int x = 0; x < 2; ++x) {
        mbar_init(bar_sfull(x), 1); mbar_init(bar_pready(x), 128); mbar_init(bar_pready2(x), 128); mbar_init(bar_pvdone(x), 1);
      }
      mbar_init(bar_alldone, 1);
      *abort_flag = 0;
      fence_barrier_init();
      fence_proxy_async();
    }
    if (use_list) {
      for (int t = lane; t < nt; t += 32) {
        const TileInfo ti = tile_info(p, te, t0 + t);
        if (t0 + t < te.n_blk && ti.nvalid == 0) set_status(p.status, FOCUS_ERR_INVALID_ARG);   // bad block index
        tlist[t] = pack_tile(ti);
      }
    }
    __syncwarp();
    if (lane < n_early) issue(lane);                             // one copy per lane
    __syncwarp();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_holder), 512);
    tmem_relinquish();
  }
  if (stager) {                                                  // query tile X at X * 32 KB, swizzled K-major
    if (my_fr < total_fr && !pos_ok) set_status(p.status, FOCUS_ERR_INVALID_ARG);
    const bool live = my_fr < total_fr;                          // rows beyond the count are staged as zeros
    const int x = qtid >> 7, rr = qtid & 127;
#pragma unroll
    for (int c = 0; c < QCH; ++c) {
      const int half = c >> 3, cc = c & 7;
      *reinterpret_cast<uint4*>(sptr + x * Q_BYTES + half * HALF_BYTES + rr * 128 + ((cc ^ (rr & 7)) << 4)) =
          live ? qv[c] : make_uint4(0, 0, 0, 0);
    }
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_holder;
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
  if (warp == 0) {
    if (lane == 0) {
      int issued = n_early;
      bool ok = true;
      if (n_early < n_loads) ok = mbar_wait(bar_full(0), 0u, abort_flag, p.status);   // K0 first (see the one-tile kernel)
      for (int q = n_early; q < n_loads && ok; ++q) {
        if (!mbar_wait(bar_empty(q % NSLOT_W), (uint32_t)((q / NSLOT_W) & 1) ^ 1u, abort_flag, p.status)) { ok = false; break; }
        issue(q);
        ++issued;
      }
      if (!ok) {
        const uint32_t first = issued > NSLOT_W ? (uint32_t)(issued - NSLOT_W) : 0u;
        for (uint32_t i = first; i < (uint32_t)issued; ++i) {
          const uint64_t t_start = global_ns();
          while (!mbar_try_wait(bar_full(i % NSLOT_W), (i / NSLOT_W) & 1u))
            if (global_ns() - t_start > WAIT_LIMIT_NS) break;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = make_idesc(TM, TN, 0);
      const uint32_t IDESC_PV = p.hd > 64 ? make_idesc(TM, HD, 1) : make_idesc(TM, 64, 1);   // head dim 64: O is 64 columns wide
      bool ok = true;
      auto wait_load = [&](int q) { return mbar_wait(bar_full(q % NSLOT_W), (uint32_t)(q / NSLOT_W) & 1u, abort_flag, p.status); };
      auto do_qk = [&](int x, int j) {                              // S_x = Q_x K_j^T (KP: the one query tile)
        const uint64_t qdesc = make_sdesc(sQ + (KP ? 0 : x) * Q_BYTES, 16, 1024);
        const uint64_t kdesc = make_sdesc(sSlot + ((2 * j) % NSLOT_W) * SLOT_BYTES, 16, 1024);
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            if (half == 1 && p.hd <= 64) continue;                   // head dim 64: one half of the contraction
            const uint64_t off = (uint64_t)((half * HALF_BYTES + ks * 32) >> 4);
            mma_ss(tmem + x * 128, qdesc + off, kdesc + off, IDESC_QK, (half | ks) ? 1u : 0u);
          }
        tc_commit(bar_sfull(x));
      };
      // O_x += P_x(j) V_j in two halves of 64 keys: the first starts while the softmax warps still work on the second
      auto do_pv = [&](int x, int j, uint32_t par, bool first) -> bool {
        const uint64_t vdesc = make_sdesc(sSlot + ((2 * j + 1) % NSLOT_W) * SLOT_BYTES, HALF_BYTES, 1024);
        if (!mbar_wait(bar_pready(x), par, abort_flag, p.status)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < TN / 32; ++ks)
          mma_ts(tmem + 256 + x * 128, tmem + x * 128 + ks * 8, vdesc + (uint64_t)(ks * (2048 >> 4)), IDESC_PV,
                 (!first || ks > 0) ? 1u : 0u);
        if (!mbar_wait(bar_pready2(x), par, abort_flag, p.status)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = TN / 32; ks < TN / 16; ++ks)
          mma_ts(tmem + 256 + x * 128, tmem + x * 128 + ks * 8, vdesc + (uint64_t)(ks * (2048 >> 4)), IDESC_PV, 1u);
        tc_commit(bar_pvdone(x));
        return true;
      };
      if (KP) {
        // key tile t belongs to warpgroup t & 1; consumption order K0, K1, V0, K2, V1, K3, ... stays inside the
        // ring window (the oldest slot still held and the newest one needed are at most four loads apart)
        ok = wait_load(0);
        if (ok) {
          tc_fence_after();
          do_qk(0, 0);
          tc_commit(bar_empty(0));
        }
        if (ok && nt > 1) {
          ok = wait_load(2);
          if (ok) {
            tc_fence_after();
            do_qk(1, 1);
            tc_commit(bar_empty(2 % NSLOT_W));
          }
        }
        for (int t = 0; t < nt && ok; ++t) {
          const int x = t & 1;
          if (!wait_load(2 * t + 1)) { ok = false; break; }          // V_t
          if (!do_pv(x, t, (uint32_t)(t >> 1) & 1u, t < 2)) { ok = false; break; }
          tc_commit(bar_empty((2 * t + 1) % NSLOT_W));
          if (t + 2 < nt) {
            if (!wait_load(2 * t + 4)) { ok = false; break; }        // K_(t+2)
            tc_fence_after();
            do_qk(x, t + 2);
            tc_commit(bar_empty((2 * t + 4) % NSLOT_W));
          }
        }
      } else {
      ok = wait_load(0);
      if (ok) {
        tc_fence_after();
        do_qk(0, 0);
        do_qk(1, 0);
        tc_commit(bar_empty(0));                                     // K_0's slot: free once both products have read it
      }
      for (int j = 0; j < nt && ok; ++j) {
        const uint32_t par = (uint32_t)j & 1u;
        if (!wait_load(2 * j + 1)) { ok = false; break; }            // V_j
        if (!do_pv(0, j, par, j == 0)) { ok = false; break; }
        if (j + 1 < nt) {
          if (!wait_load(2 * j + 2)) { ok = false; break; }          // K_(j+1)
          tc_fence_after();
          do_qk(0, j + 1);
        }
        if (!do_pv(1, j, par, j == 0)) { ok = false; break; }
        tc_commit(bar_empty((2 * j + 1) % NSLOT_W));                 // V_j
        if (j + 1 < nt) {
          do_qk(1, j + 1);
          tc_commit(bar_empty((2 * j + 2) % NSLOT_W));               // K_(j+1)
        }
      }
      }
      tc_commit(bar_alldone);
    }
  }
    // tail of the first warpgroup, inside its own register-budget region: release TMEM, take part in the barriers of
    // the merge (registers given away above are not asked back: a late setmaxnreg.inc never returned on this part)
    tc_fence_before();
    asm volatile("bar.sync 0;" ::: "memory");
    if (warp == 1) {
      __syncwarp();
      tmem_dealloc(tmem, 512);
    }
    if (p.n_splits > 1) cluster_merge<TMQ, 256>(p, g, mt, total_fr, split, sSlot, -1);
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    const int x = (warp - 4) >> 2;                                   // query tile of this softmax warp
    const int rq = warp & 3;
    const int row = rq * 32 + lane;                                  // row inside the 128-row tile
    const uint32_t lane_off = (uint32_t)(rq * 32) << 16;
    const uint32_t ts = tmem + lane_off + x * 128;
    const uint32_t to = tmem + lane_off + 256 + x * 128;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    const int nt_x = KP ? (nt - x + 1) / 2 : nt;                     // key tiles of this warpgroup
    for (int idx = 0; idx < nt_x; ++idx) {
      if (!__all_sync(0xffffffffu, mbar_wait(bar_sfull(x), (uint32_t)idx & 1u, abort_flag, p.status))) { ok = false; break; }
      tc_fence_after();
      uint32_t sreg[128];
      TC_LD32(ts, (sreg + 0));
      TC_LD32(ts + 32, (sreg + 32));
      TC_LD32(ts + 64, (sreg + 64));
      TC_LD32(ts + 96, (sreg + 96));
      tc_wait_ld();
      const TileInfo ti = get_tile(KP ? 2 * idx + x : idx);
      float tmax = -INFINITY;
      if (ti.kind == 0 && ti.nvalid == TN) {
        float t4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains instead of one of 128
#pragma unroll
        for (int c = 0; c < 128; c += 8) {
          t4[0] = fmax3(t4[0], __uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1]));
          t4[1] = fmax3(t4[1], __uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3]));
          t4[2] = fmax3(t4[2], __uint_as_float(sreg[c + 4]), __uint_as_float(sreg[c + 5]));
          t4[3] = fmax3(t4[3], __uint_as_float(sreg[c + 6]), __uint_as_float(sreg[c + 7]));
        }
        tmax = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
      } else if (ti.kind == 0) {
#pragma unroll
        for (int c = 0; c < 128; ++c) {
          const float v = c < ti.nvalid ? __uint_as_float(sreg[c]) : -INFINITY;
          sreg[c] = __float_as_uint(v);
          tmax = fmaxf(tmax, v);
        }
      } else {
        const uint32_t* mk = reinterpret_cast<const uint32_t*>(p.sink_mask + (size_t)g * p.ns_pad + ti.start);
#pragma unroll
        for (int c4 = 0; c4 < 32; ++c4) {
          const uint32_t mword = __ldg(mk + c4);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int c = c4 * 4 + e;
            const float v = ((mword >> (8 * e)) & 0xffu) ? __uint_as_float(sreg[c]) : -INFINITY;
            sreg[c] = __float_as_uint(v);
            tmax = fmaxf(tmax, v);
          }
        }
      }
      tmax *= p.scale_log2;
      float alpha = 1.f;
      bool rescale = false;
      if (tmax > m_ref + RESCALE_THRESHOLD) {
        if (m_ref != -INFINITY) {
          alpha = ex2(m_ref - tmax);
          rescale = true;
        }
        m_ref = tmax;
      }
      const float mneg = m_ref == -INFINITY ? 0.f : -m_ref;
      // sfull(idx) implies that every earlier product of this tile, P V of key tile idx-1 included, has completed
      if (idx > 0 && __any_sync(0xffffffffu, rescale)) {
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t oreg[32];
          TC_LD32(to + cb * 32, oreg);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) oreg[c] = __float_as_uint(__uint_as_float(oreg[c]) * alpha);
          TC_ST32(to + cb * 32, oreg);
        }
      }
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {                               // 32 keys at a time: exponentials, bf16 P, row sum
        uint32_t preg[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int c = ch * 32 + 2 * i;
          float x0, x1;
          ffma2(x0, x1, __uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1]), p.scale_log2, p.scale_log2, mneg, mneg);
          const float p0 = ex2(x0), p1 = ex2(x1);
          preg[i] = pack_bf16(p0, p1);
          fadd2(acc[(i & 1) * 2], acc[(i & 1) * 2 + 1], acc[(i & 1) * 2], acc[(i & 1) * 2 + 1], p0, p1);
        }
        TC_ST16(ts + ch * 16, preg);
        if (ch == 1) {
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(bar_pready(x));
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_pready2(x));
      l = l * alpha + ((acc[0] + acc[1]) + (acc[2] + acc[3]));
    }
    if (ok && nt_x > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar_pvdone(x), (uint32_t)(nt_x - 1) & 1u, abort_flag, p.status));
    if (KP) {
      // Merge of the two warpgroups' halves.  Both accumulators are complete once every MMA of the CTA has retired;
      // the (reference max, row sum) pairs cross through shared memory (over the K/V ring, idle by then).
      ok = ok && __all_sync(0xffffffffu, mbar_wait(bar_alldone, 0u, abort_flag, p.status));
      tc_fence_after();
      float2* xch = reinterpret_cast<float2*>(ps + TMQ * PROW + 2 * TMQ);
      if (ok) xch[x * TM + row] = make_float2(nt_x > 0 ? m_ref : -INFINITY, nt_x > 0 ? l : 0.f);
      asm volatile("bar.sync 1, 256;" ::: "memory");                 // the eight softmax warps (taken on every path)
      if (ok) {
        const float2 ea = xch[row], eb = xch[TM + row];
        float m = -INFINITY;
        if (ea.y > 0.f) m = ea.x;
        if (eb.y > 0.f) m = fmaxf(m, eb.x);
        const float wa = ea.y > 0.f ? ex2(ea.x - m) : 0.f, wb = eb.y > 0.f ? ex2(eb.x - m) : 0.f;
        const float tot = wa * ea.y + wb * eb.y;
        const int fr = mt * TMQ + row;
        const bool valid = fr < total_fr;
        const int qr = valid ? fr / p.hpg : 0, hh = valid ? fr % p.hpg : 0;
        const float inv = p.n_splits == 1 ? (tot > 0.f ? 1.f / tot : 0.f) : 1.f;
        const float fa = wa * inv, fb = wb * inv;
        const uint32_t toa = tmem + lane_off + 256, tob = tmem + lane_off + 384;
        __nv_bfloat16* orow = p.O + ((size_t)qr * p.H + (size_t)(g * p.hpg + hh)) * p.hd;
        float* prow = ps + row * PROW;
#pragma unroll
        for (int cb = 2 * x; cb < 2 * x + 2; ++cb) {                 // this warpgroup's 64 output columns
          uint32_t oa[32], ob[32];
          TC_LD32(toa + cb * 32, oa);
          if (nt > 1) TC_LD32(tob + cb * 32, ob);                    // with one key tile O_B was never written
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            float v = __uint_as_float(oa[c]) * fa;
            if (nt > 1 && fb > 0.f) v = fmaf(__uint_as_float(ob[c]), fb, v);
            oa[c] = __float_as_uint(v);
          }
          if (valid) {
            if (p.n_splits == 1) {
#pragma unroll
              for (int c = 0; c < 32; c += 8) {
                uint4 v;
                v.x = pack_bf16(__uint_as_float(oa[c + 0]), __uint_as_float(oa[c + 1]));
                v.y = pack_bf16(__uint_as_float(oa[c + 2]), __uint_as_float(oa[c + 3]));
                v.z = pack_bf16(__uint_as_float(oa[c + 4]), __uint_as_float(oa[c + 5]));
                v.w = pack_bf16(__uint_as_float(oa[c + 6]), __uint_as_float(oa[c + 7]));
                if (cb * 32 < p.hd) *reinterpret_cast<uint4*>(orow + cb * 32 + c) = v;
              }
            } else {
#pragma unroll
              for (int c = 0; c < 32; c += 4)
                *reinterpret_cast<uint4*>(prow + cb * 32 + c) = make_uint4(oa[c], oa[c + 1], oa[c + 2], oa[c + 3]);
            }
          }
        }
        if (valid && x == 0) {
          if (p.n_splits == 1) {
            if (p.lse) p.lse[(size_t)(g * p.hpg + hh) * p.lse_stride + qr] = (m + log2f(tot)) * 0.6931471805599453f;
          } else {
            ps[TMQ * PROW + 2 * row] = m; ps[TMQ * PROW + 2 * row + 1] = tot;
          }
        }
      }
    } else if (ok) {
      tc_fence_after();
      const int trow = x * 128 + row;                                // row inside the 256-row CTA tile
      const int fr = mt * TMW + trow;
      const bool valid = fr < total_fr;
      if (p.n_splits == 1) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const int qr = valid ? fr / p.hpg : 0, hh = valid ? fr % p.hpg : 0;
        __nv_bfloat16* orow = p.O + ((size_t)qr * p.H + (size_t)(g * p.hpg + hh)) * p.hd;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t oreg[32];
          TC_LD32(to + cb * 32, oreg);
          tc_wait_ld();
          if (valid) {
#pragma unroll
            for (int c = 0; c < 32; c += 8) {
              uint4 v;
              v.x = pack_bf16(__uint_as_float(oreg[c + 0]) * inv, __uint_as_float(oreg[c + 1]) * inv);
              v.y = pack_bf16(__uint_as_float(oreg[c + 2]) * inv, __uint_as_float(oreg[c + 3]) * inv);
              v.z = pack_bf16(__uint_as_float(oreg[c + 4]) * inv, __uint_as_float(oreg[c + 5]) * inv);
              v.w = pack_bf16(__uint_as_float(oreg[c + 6]) * inv, __uint_as_float(oreg[c + 7]) * inv);
              if (cb * 32 < p.hd) *reinterpret_cast<uint4*>(orow + cb * 32 + c) = v;
            }
          }
        }
        if (valid && p.lse)
          p.lse[(size_t)(g * p.hpg + hh) * p.lse_stride + qr] = (m_ref + log2f(l)) * 0.6931471805599453f;
      } else if (__all_sync(0xffffffffu, mbar_wait(bar_alldone, 0u, abort_flag, p.status)) &&
                 __any_sync(0xffffffffu, valid)) {
        // cluster mode: partial into own shared memory, which overlays the K/V ring -- the other query tile's last
        // P V product may still be reading its V tile there, hence the wait for every MMA of the CTA
        float* prow = ps + trow * PROW;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t oreg[32];
          TC_LD32(to + cb * 32, oreg);
          tc_wait_ld();
          if (valid) {
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              *reinterpret_cast<uint4*>(prow + cb * 32 + c) = make_uint4(oreg[c], oreg[c + 1], oreg[c + 2], oreg[c + 3]);
          }
        }
        if (valid) { ps[TMW * PROW + 2 * trow] = m_ref; ps[TMW * PROW + 2 * trow + 1] = l; }
      }
    }
    // tail of the softmax warpgroups (kept inside their register-budget region): they do the split merge
    tc_fence_before();
    asm volatile("bar.sync 0;" ::: "memory");
    if (p.n_splits > 1) cluster_merge<TMQ, 256>(p, g, mt, total_fr, split, sSlot, (int)threadIdx.x - 128);
  }
}

// Stand-alone merge (used when there are more query tiles than arrival counters): out = sum_s 2^(m_s - m) O_s / sum_s 2^(m_s - m) l_s, one warp per stacked row.
__global__ void __launch_bounds__(256)
attn_combine_kernel(const float* __restrict__ part_O, const float* __restrict__ part_ml, int n_splits, int n_mtiles,
                    int hpg, int H, const int32_t* q_rows, const int32_t* n_rows, int rows_bound, int n_q,
                    __nv_bfloat16* __restrict__ O, float* __restrict__ lse, int lse_stride, int hd) {
  const int lane = threadIdx.x & 31;
  const int wrow = blockIdx.x * 8 + (threadIdx.x >> 5);        // global stacked-row slot: tile * 128 + row
  const int tile = wrow / TM, row = wrow % TM;
  const int g = tile / n_mtiles, mt = tile % n_mtiles;
  const int nrows = q_rows ? min(max(*n_rows, 0), rows_bound) : n_q;
  const int fr = mt * TM + row;
  if (fr >= nrows * hpg) return;
  float m = -INFINITY;
  for (int s = 0; s < n_splits; ++s) {
    const float* ml = part_ml + ((size_t)(tile * n_splits + s) * TM + row) * 2;
    if (ml[1] > 0.f) m = fmaxf(m, ml[0]);
  }
  float tot = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < n_splits; ++s) {
    const size_t base = (size_t)(tile * n_splits + s) * TM + row;
    const float ls = part_ml[base * 2 + 1];
    if (!(ls > 0.f)) continue;
    const float wgt = exp2f(part_ml[base * 2] - m);
    tot += wgt * ls;
    const float4 o = *reinterpret_cast<const float4*>(part_O + base * HD + lane * 4);
    acc.x += wgt * o.x; acc.y += wgt * o.y; acc.z += wgt * o.z; acc.w += wgt * o.w;
  }
  const float inv = tot > 0.f ? 1.f / tot : 0.f;
  const int qr = fr / hpg, hh = fr % hpg;
  __nv_bfloat16* orow = O + ((size_t)qr * H + (size_t)(g * hpg + hh)) * hd + lane * 4;
  uint2 v;
  v.x = pack_bf16(acc.x * inv, acc.y * inv);
  v.y = pack_bf16(acc.z * inv, acc.w * inv);
  if (lane * 4 < hd) *reinterpret_cast<uint2*>(orow) = v;
  if (lse && lane == 0) lse[(size_t)(g * hpg + hh) * lse_stride + qr] = (m + log2f(tot)) * 0.6931471805599453f;
}

// Gathers the sink tokens' K and V rows into compact, zero-padded per-KV-head tiles and builds the
// column mask: attend column s iff the token is kept for this head's group, is valid and is a prompt token
// (response tokens are attended through the response tiles; every key is counted once).
__global__ void __launch_bounds__(256)
sink_gather_kernel(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V, long long kv_stride_tok,
                   long long kv_stride_head, const int32_t* __restrict__ sink_idx, const uint8_t* __restrict__ sink_keep,
                   int n_sink, int ns_pad, int group_stride, int M, int L, __nv_bfloat16* __restrict__ gK,
                   __nv_bfloat16* __restrict__ gV, uint8_t* __restrict__ mask, int32_t* status, int hd) {
  const int g = blockIdx.y;
  const int s = blockIdx.x * 16 + (threadIdx.x >> 4), c = threadIdx.x & 15;
  if (s >= ns_pad || c * 8 >= hd) return;
  uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
  uint8_t mk = 0;
  if (s < n_sink) {
    const int j = sink_idx[s];
    if (j < 0 || j >= L) {
      if (c == 0) set_status(status, FOCUS_ERR_INVALID_ARG);
    } else {
      const size_t off = (size_t)g * kv_stride_head + (size_t)j * kv_stride_tok + c * 8;
      kv = __ldg(reinterpret_cast<const uint4*>(K + off));
      vv = __ldg(reinterpret_cast<const uint4*>(V + off));
      mk = (j < M && sink_keep[(size_t)g * group_stride * n_sink + s]) ? 1 : 0;
    }
  }
  const size_t o = ((size_t)g * ns_pad + s) * hd + c * 8;
  *reinterpret_cast<uint4*>(gK + o) = kv;
  *reinterpret_cast<uint4*>(gV + o) = vv;
  if (c == 0) mask[(size_t)g * ns_pad + s] = mk;
}

int pick_splits(const focus_ctx* ctx, int base_ctas, int max_tiles) {
  int s = ctx->sm_count / (base_ctas > 0 ? base_ctas : 1);
  if (s < 1) s = 1;
  const int cap = max_tiles / 2 > 1 ? max_tiles / 2 : 1;
  if (s > cap) s = cap;
  return s > 8 ? 8 : s;                      // at most 8 splits: they form one (portable-size) thread-block cluster
}

// How many clusters of `n` CTAs of this kernel (one CTA per SM, maximum shared memory) can be resident at once on
// this device.  It depends on how the enabled SMs are spread over the GPCs, which differs from chip to chip.
template <typename K>
static int cluster_capacity(K kernel, int n, int threads, int smem) {
  cudaLaunchConfig_t qc = {};
  qc.gridDim = dim3(n, n, 1); qc.blockDim = dim3(threads, 1, 1); qc.dynamicSmemBytes = smem;
  cudaLaunchAttribute qa[1];
  qa[0].id = cudaLaunchAttributeClusterDimension;
  qa[0].val.clusterDim.x = 1; qa[0].val.clusterDim.y = n; qa[0].val.clusterDim.z = 1;
  qc.attrs = qa; qc.numAttrs = 1;
  int n_clusters = 0;
  const cudaError_t e = cudaOccupancyMaxActiveClusters(&n_clusters, kernel, &qc);
  if (e != cudaSuccess) { cudaGetLastError(); return 0; }
  return n_clusters;
}

template <typename K>
static focus_status launch_ex(K kernel, dim3 grid, int threads, int smem, int cluster_y, bool pdl, cudaStream_t st,
                              const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, const CUtensorMap& d,
                              const TcParams& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = dim3(threads, 1, 1); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (cluster_y > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = 1; at[na].val.clusterDim.y = cluster_y; at[na].val.clusterDim.z = 1;
    ++na;
  }
  if (pdl) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at; cfg.numAttrs = na;
  if (cudaLaunchKernelEx(&cfg, kernel, a, b, c, d, p) != cudaSuccess) {
    cudaGetLastError();
    return FOCUS_ERR_CUDA;
  }
  return FOCUS_OK;
}

}  // namespace

bool attn_tc_supported(const focus_ctx* ctx, const AttnArgs& a) {
  return ctx->encode_tiled != nullptr && a.sh.dtype == FOCUS_BF16 && (a.sh.head_dim == HD || a.sh.head_dim == 64) && a.O != nullptr &&
         (a.sh.n_q_heads / a.sh.n_kv_heads) <= TM && a.sh.L >= 1;
}

size_t attn_tc_workspace(const focus_shape* s, int n_q, int max_blocks, int n_sink) {
  const size_t ns_pad = ((size_t)n_sink + TN - 1) / TN * TN;
  const size_t gather = 2 * (size_t)s->n_kv_heads * ns_pad * HD * 2 + (size_t)s->n_kv_heads * ns_pad + 1024;
  const int hpg = s->n_q_heads / s->n_kv_heads;
  const size_t mtiles = ((size_t)n_q * hpg + TM - 1) / TM;
  const size_t ctas = mtiles * s->n_kv_heads;
  const size_t part = (ctas < 160 ? 320 : ctas) * ((size_t)TM * HD * 4 + TM * 8) + 1024;
  return gather + part;
}

focus_status launch_attn_tc(focus_ctx* ctx, const AttnArgs& a, cudaStream_t st) {
  WsAlloc ws(ctx);
  return launch_attn_tc_ws(ctx, a, ws, nullptr, st);
}

// `pre` non-NULL: the sink rows and the column mask were already gathered into it by the caller (taken from `ws`).
focus_status launch_attn_tc_ws(focus_ctx* ctx, const AttnArgs& a, WsAlloc& ws, const SinkGather* pre, cudaStream_t st) {
  const focus_shape& sh = a.sh;
  const int Hkv = sh.n_kv_heads, hpg = sh.n_q_heads / Hkv;
  const long long stacked = (long long)a.max_rows * hpg;            // stacked query rows per KV head (host bound)
  if (stacked == 0) return FOCUS_OK;
  const int ns_pad = a.dense ? 0 : (a.n_sink + TN - 1) / TN * TN;
  const int n_resp = a.dense ? (sh.L + TN - 1) / TN : (sh.L - sh.M + TN - 1) / TN;
  // 64-token KV blocks: two selected blocks share a 128-key tile
  const bool pair = !a.dense && sh.kv_block == 64;
  const int max_tiles = a.dense ? n_resp : (pair ? (a.max_blocks + 1) / 2 : a.max_blocks) + ns_pad / TN + n_resp;
  bool& attr_set = ctx->ls.attn_attr_set;
  if (!attr_set) {
    if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(attn_tc_wide_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES_W) != cudaSuccess ||
        cudaFuncSetAttribute(attn_tc_wide_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES_W) != cudaSuccess)
      return FOCUS_ERR_CUDA;
    attr_set = true;
  }
  // resident-cluster capacity per cluster size (-1 = not asked yet): a launch whose clusters do not all fit at once
  // would run in two waves, so such launches fall back to the merge through global memory (narrow kernel) or to
  // the narrow kernel (wide kernel)
  int* cluster_cap = ctx->ls.cluster_cap;          // stored as capacity + 1: 0 means "not asked yet"
  int* cluster_cap_w = ctx->ls.cluster_cap_w;
  // two query tiles per CTA when a KV head has at least 256 stacked rows (tensor-bound regime)
  bool wide = stacked >= TMW && !ctx->no_wide;
  int n_mtiles = 0, base = 0, n_splits = 1;
  if (wide) {
    n_mtiles = (int)((stacked + TMW - 1) / TMW);
    base = n_mtiles * Hkv;
    n_splits = pick_splits(ctx, base, max_tiles);
    if (n_splits > 1) {
      if (cluster_cap_w[n_splits] == 0)
        cluster_cap_w[n_splits] = cluster_capacity(attn_tc_wide_kernel<false>, n_splits, NTHREADS_W, SMEM_BYTES_W) + 1;
      if (cluster_cap_w[n_splits] - 1 < base) wide = false;           // its splits merge through a cluster only
    }
    // it pays from about 24 key tiles per CTA upward (measured at 256 rows, 32 heads: 32 tiles per CTA 85 us against
    // 87 us for the key-pair form, 17 to 19 tiles per CTA 3 to 12 % slower than it); below that the one-tile forms,
    // which need fewer or no key splits, win
    if (max_tiles / n_splits < WIDE_MIN_TILES) wide = false;
  }
  // key-pair form: one query tile per CTA, two softmax warpgroups on alternating key tiles.  For query sets with
  // enough rows per tile to be bound by the exponentials (not by HBM) that the two-tile form does not take.
  bool kpair = false;
  if (!wide) {
    n_mtiles = (int)((stacked + TM - 1) / TM);
    base = n_mtiles * Hkv;
    n_splits = pick_splits(ctx, base, max_tiles);
    if (!ctx->no_wide && stacked >= KP_MIN_ROWS && max_tiles / n_splits >= KP_MIN_TILES &&
        (n_splits == 1 || ctx->merge_mode == 0)) {
      kpair = true;
      if (n_splits > 1) {                                                // its splits merge through a cluster only
        int* cap = ctx->ls.cluster_cap_k;
        if (cap[n_splits] == 0)
          cap[n_splits] = cluster_capacity(attn_tc_wide_kernel<true>, n_splits, NTHREADS_W, SMEM_BYTES_W) + 1;
        if (cap[n_splits] - 1 < base) kpair = false;
      }
    }
  }
  const bool wg3 = wide || kpair;                                        // three-warpgroup kernel (either form)

  __nv_bfloat16* gK = nullptr; __nv_bfloat16* gV = nullptr; uint8_t* mask = nullptr;
  if (ns_pad > 0) {
    if (pre) {
      gK = pre->gK; gV = pre->gV; mask = pre->mask;
    } else {
      gK = ws.get<__nv_bfloat16>((size_t)Hkv * ns_pad * HD);
      gV = ws.get<__nv_bfloat16>((size_t)Hkv * ns_pad * HD);
      mask = ws.get<uint8_t>((size_t)Hkv * ns_pad);
    }
  }
  bool use_cluster = false;
  if (n_splits > 1 && !wg3 && ctx->merge_mode == 0) {
    // the largest split count (not above the one wanted) whose clusters are all resident at once; if even two-CTA
    // clusters do not fit, keep the wanted count and merge through global memory
    for (int sp = n_splits; sp >= 2; --sp) {
      if (cluster_cap[sp] == 0) cluster_cap[sp] = cluster_capacity(attn_tc_kernel, sp, NTHREADS, SMEM_BYTES) + 1;
      if (cluster_cap[sp] - 1 >= base) { n_splits = sp; use_cluster = true; break; }
    }
    if (getenv("FOCUS_LOG")) fprintf(stderr, "[focus] attn: base %d splits %d cluster %d\n", base, n_splits, (int)use_cluster);
  }
  if (wg3) use_cluster = n_splits > 1;
  float* part_O = nullptr; float* part_ml = nullptr;
  if (n_splits > 1 && !use_cluster && !wg3) {
    part_O = ws.get<float>((size_t)base * n_splits * TM * HD);
    part_ml = ws.get<float>((size_t)base * n_splits * TM * 2);
  }
  if (!ws.ok) return FOCUS_ERR_WORKSPACE_TOO_SMALL;

  // head dim 64: the maps' inner extent is 64, so the copy of a tile's upper 64 columns lies wholly outside the
  // tensor and arrives as zeros -- the kernels run their 128-wide geometry on operands padded for free
  const int hd = sh.head_dim;
  CUtensorMap tmK, tmV, tmSK, tmSV;
  const int box_rows = pair ? 64 : TN;
  if (!encode_kv_map(ctx->encode_tiled, &tmK, a.K, hd, sh.L, Hkv, sh.kv_stride_tok, sh.kv_stride_head, 64, box_rows) ||
      !encode_kv_map(ctx->encode_tiled, &tmV, a.V, hd, sh.L, Hkv, sh.kv_stride_tok, sh.kv_stride_head, 64, box_rows))
    return FOCUS_ERR_INVALID_ARG;
  if (ns_pad > 0) {
    if (!encode_kv_map(ctx->encode_tiled, &tmSK, gK, hd, ns_pad, Hkv, hd, (long long)ns_pad * hd, 64, TN) ||
        !encode_kv_map(ctx->encode_tiled, &tmSV, gV, hd, ns_pad, Hkv, hd, (long long)ns_pad * hd, 64, TN))
      return FOCUS_ERR_CUDA;
    if (!pre) {
      dim3 gg((ns_pad + 15) / 16, Hkv);
      sink_gather_kernel<<<gg, 256, 0, st>>>((const __nv_bfloat16*)a.K, (const __nv_bfloat16*)a.V, sh.kv_stride_tok,
                                             sh.kv_stride_head, a.sink_idx, a.sink_keep, a.n_sink, ns_pad,
                                             a.group_stride, sh.M, sh.L, gK, gV, mask, ctx->d_status, hd);
      FOCUS_CHECK_LAUNCH();
    }
  } else {
    tmSK = tmK; tmSV = tmV;
  }

  TcParams p;
  p.Q = (const __nv_bfloat16*)a.Q; p.O = (__nv_bfloat16*)a.O; p.lse = a.lse;
  p.q_rows = a.q_rows; p.n_rows = a.n_rows; p.block_idx = a.block_idx; p.block_cnt = a.block_cnt;
  p.sink_mask = mask; p.part_O = part_O; p.part_ml = part_ml;
  p.cluster = use_cluster ? 1 : 0;
  p.pair = pair ? 1 : 0;
  p.hd = hd;
  // K/V ring slots the one-tile kernel keeps in flight: a short key loop is a chain of latencies and wants the tile it
  // needs next delivered first (every copy in flight takes its share of the CTA's bandwidth); a long one wants one
  // more slot to ride out the jitter.  Measured, I_active rows, 128 CTAs: 5-6 tiles per CTA 24.9 us with six slots,
  // 23.2 with four, 22.9 with three; 64 tiles per CTA (dense) 87.0 / 85.7 / 87.7 us; 33 tiles 61.1 / 59.4 / 61.1.
  p.ring = max_tiles / n_splits >= 12 ? RING_LONG : RING_SHORT;
  // 1: called right after the selection kernel of a fused sparse layer (pre-gathered sinks); 2: predecessor unknown
  p.pdl = ctx->no_pdl ? 0 : ((pre != nullptr && !wg3) ? 1 : 2);
  p.counters = (n_splits > 1 && !use_cluster && !wg3 && ctx->merge_mode != 2 && base <= FOCUS_N_COUNTERS && (size_t)(TM * n_splits + TM) * 4 <= (size_t)NSLOT * SLOT_BYTES)
                   ? ctx->d_counters : nullptr;
  p.q_stride_row = sh.q_stride_row; p.q_stride_head = sh.q_stride_head;
  p.q_base = a.q_base; p.n_q = a.n_q; p.rows_bound = a.max_rows; p.L = sh.L; p.M = sh.M; p.H = sh.n_q_heads;
  p.Hkv = Hkv; p.hpg = hpg; p.B = sh.kv_block; p.nb = shape_nb(&sh); p.dense = a.dense;
  p.group_stride = a.group_stride; p.max_blocks = a.max_blocks; p.n_sink = a.n_sink; p.ns_pad = ns_pad;
  p.n_mtiles = n_mtiles; p.n_splits = n_splits; p.lse_stride = a.lse_stride;
  p.scale_log2 = a.scale * 1.4426950408889634f;
  p.status = ctx->d_status;

  ctx->last_attn_variant = wide ? 3 : (kpair ? 4 : 2);
  if (wide) {
    focus_status ls = launch_ex(attn_tc_wide_kernel<false>, dim3(base, n_splits, 1), NTHREADS_W, SMEM_BYTES_W, n_splits, p.pdl != 0, st,
                                tmK, tmV, tmSK, tmSV, p);
    if (ls != FOCUS_OK) return ls;
  } else if (kpair) {
    focus_status ls = launch_ex(attn_tc_wide_kernel<true>, dim3(base, n_splits, 1), NTHREADS_W, SMEM_BYTES_W, n_splits, p.pdl != 0, st,
                                tmK, tmV, tmSK, tmSV, p);
    if (ls != FOCUS_OK) return ls;
  } else {
    focus_status ls = launch_ex(attn_tc_kernel, dim3(base, n_splits, 1), NTHREADS, SMEM_BYTES, use_cluster ? n_splits : 1,
                                p.pdl != 0, st, tmK, tmV, tmSK, tmSV, p);
    if (ls != FOCUS_OK) return ls;
  }
  FOCUS_CHECK_LAUNCH();
  if (n_splits > 1 && !p.counters && !use_cluster && !wg3) {
    const int rows_total = base * TM;
    attn_combine_kernel<<<rows_total / 8, 256, 0, st>>>(part_O, part_ml, n_splits, n_mtiles, hpg, sh.n_q_heads,
                                                        a.q_rows, a.n_rows, a.max_rows, a.n_q,
                                                        (__nv_bfloat16*)a.O, a.lse, a.lse_stride, hd);
    FOCUS_CHECK_LAUNCH();
  }
  return FOCUS_OK;
}

// ---- self-test of the bounded waits -------------------------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(unsigned long long limit_ns, int32_t* status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncwarp();
  // nobody arrives: the wait must give up after limit_ns, raise the flag and the status word, and return false
  mbar_wait(b, 0u, &abort_flag, status, limit_ns);
}
}  // namespace

extern "C" focus_status focus_selftest_bounded_wait(focus_ctx* ctx, int32_t limit_us, focus_stream stream) {
  if (!ctx || limit_us < 1 || limit_us > 100000) return FOCUS_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((unsigned long long)limit_us * 1000ull, ctx->d_status);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}
