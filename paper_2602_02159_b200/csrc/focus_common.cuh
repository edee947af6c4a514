// Shared host/device helpers of libfocus (internal; the public ABI is include/focus.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include "focus.h"

struct focus_ctx {
  int device;
  int sm_count;
  char* ws;            // workspace (device)
  size_t ws_bytes;
  int32_t* d_status;   // device status word: 0 = clean, else first anomaly's focus_status code
  int32_t* d_counters; // FOCUS_N_COUNTERS arrival counters for split merges; zero between launches
  int force_simt;
  int last_attn_variant;   // 0 none yet, 1 SIMT, 2 tensor-core 128-row tiles, 3 tensor-core 256-row tiles, 4 key-pair form
  int no_pdl;          // 1: never launch the attention kernel as a programmatic dependent (focus_set_option)
  int no_wide;         // 1: never use the three-warpgroup attention kernels (focus_set_option)
  int merge_mode;      // split merge of the one-tile kernel: 0 automatic (cluster where it fits), 1 never a cluster (arrival
                       // counters), 2 neither (separate combine kernel); tests use 1 and 2 to reach the fallbacks
  void* encode_tiled;  // cuTensorMapEncodeTiled, resolved through the runtime (no libcuda link)
  // launch state that belongs to the device (function attributes, occupancy answers): kept per context, since a
  // process may hold contexts on several devices.  Zero-initialised by focus_create.
  struct LaunchState {
    bool attn_attr_set, select_attr_set, topn_attr_set;
    int sink_attr_smem;
    int cluster_cap[9], cluster_cap_w[9], cluster_cap_k[9];   // co-resident clusters per cluster size, value + 1 (0 = not asked yet)
    int select_cluster;                        // 0 not tried, 1 works, 2 the cluster launch was refused once
  } ls;
};

constexpr int FOCUS_N_COUNTERS = 4096;

// Bump allocator over the context workspace; one per API call.
struct WsAlloc {
  char* base;
  size_t cap, off;
  bool ok;
  explicit WsAlloc(focus_ctx* c) : base(c->ws), cap(c->ws_bytes), off(0), ok(true) {}
  template <typename T>
  T* get(size_t n) {
    size_t bytes = (n * sizeof(T) + 255) & ~size_t(255);
    if (off + bytes > cap) { ok = false; return nullptr; }
    T* p = reinterpret_cast<T*>(base + off);
    off += bytes;
    return p;
  }
};

// Every kernel launch of the library goes through this macro: it counts the launch and maps a failed
// launch to FOCUS_ERR_CUDA.
extern unsigned long long g_focus_launches;
// One NVTX range per public compute call (host side, around the enqueue): a profiler attached to the process can
// filter or group launches by stage (ncu: --nvtx --nvtx-include "focus_find_sinks/").  NVTX is header-only and costs a
// call through a null hook when no tool is attached.
struct FocusStageRange {
  explicit FocusStageRange(const char* name) { nvtxRangePushA(name); }
  ~FocusStageRange() { nvtxRangePop(); }
  FocusStageRange(const FocusStageRange&) = delete;
  FocusStageRange& operator=(const FocusStageRange&) = delete;
};
#define FOCUS_STAGE(name) FocusStageRange focus_stage_range_(name)

#define FOCUS_CHECK_LAUNCH()                                      \
  do {                                                            \
    ++g_focus_launches;                                           \
    if (cudaGetLastError() != cudaSuccess) return FOCUS_ERR_CUDA; \
  } while (0)

static inline bool shape_ok_basic(const focus_shape* s) {
  if (!s) return false;
  if (s->L <= 0 || s->M < 0 || s->M > s->L) return false;
  if (s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->n_q_heads % s->n_kv_heads) return false;
  if (s->dtype != FOCUS_F32 && s->dtype != FOCUS_BF16) return false;
  if (s->kv_block <= 0) return false;
  if (s->q_stride_row < s->head_dim || s->q_stride_head < s->head_dim) return false;
  if (s->kv_stride_tok < s->head_dim || s->kv_stride_head < s->head_dim) return false;
  if ((s->q_stride_row | s->q_stride_head | s->kv_stride_tok | s->kv_stride_head) & 7) return false;
  return true;
}
// Vector loads and TMA copies need 16-byte aligned tensors: checked on the host, a misaligned address on the device
// would fault.  NULL counts as aligned (optional arguments).
static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
template <typename... P>
static inline bool all_aligned16(P... p) { return (aligned16(p) && ...); }
static inline bool shape_supported(const focus_shape* s) {
  return (s->head_dim == 64 || s->head_dim == 128) && (s->kv_block == 64 || s->kv_block == 128);
}
static inline float shape_scale(const focus_shape* s) {
  return s->softmax_scale != 0.f ? s->softmax_scale : 1.0f / sqrtf((float)s->head_dim);
}
static inline int shape_nb(const focus_shape* s) { return (s->M + s->kv_block - 1) / s->kv_block; }

#ifdef __CUDACC__
__device__ __forceinline__ void set_status(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }

// Last statement of a kernel whose outputs a later kernel of this library reads ahead of its dependency wait (index
// lists, pooled keys, refreshed cache rows).  A programmatic dependent may start once every CTA of its predecessor has
// exited, which is not yet the point where the predecessor's writes are guaranteed visible; with this fence every
// thread's writes are visible before its CTA can exit.
__device__ __forceinline__ void publish_outputs() { __threadfence(); }

// Order-preserving map float -> uint32 (larger float => larger key).  NaN ranks below everything;
// -0 and +0 compare equal.
__device__ __forceinline__ uint32_t float_key(float x) {
  if (x != x) return 0u;
  if (x == 0.f) x = 0.f;
  uint32_t u = __float_as_uint(x);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return u == 0u ? 1u : u;   // keep 0 for NaN only (~0xFFFFFFFF is a NaN pattern anyway)
}

// Inverse of float_key: the float a key came from (NaN for key 0; -0 comes back as +0).
__device__ __forceinline__ float key_to_float(uint32_t k) {
  if (k == 0u) return __uint_as_float(0x7FC00000u);
  return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

__device__ __forceinline__ float load_as_float(const float* p) { return *p; }
__device__ __forceinline__ float load_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// Exclusive prefix sum over the thread block of one int per thread; returns the exclusive prefix and the
// block total through `total`.  `warp_tot` is shared scratch of at least 33 ints.  All threads must call.
__device__ __forceinline__ int block_excl_scan(int v, int* warp_tot, int& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();   // protect warp_tot from a previous call's readers
  if (lane == 31) warp_tot[wid] = x;
  __syncthreads();
  if (wid == 0) {
    int t = lane < nw ? warp_tot[lane] : 0;
    int s = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s += y;
    }
    if (lane < nw) warp_tot[lane] = s - t;
    if (lane == 31) warp_tot[32] = s;
  }
  __syncthreads();
  total = warp_tot[32];
  return warp_tot[wid] + x - v;
}
#endif

// ---- internal launchers (defined in the .cu files) -------------------------------------------
// Marks in sel[0..n) the C largest of the order-preserving keys key[0..n) (shared memory), equal keys taken in index
// order: the key T of the C-th largest element is found by an 8-bit radix descent (four 256-bin histograms), then
// keys > T are marked and keys == T in index order until the quota is filled.  Work per thread is O(n / threads)
// per pass, against O(n) for rank-by-counting.  Called by every thread of the block; hist: 258 ints, scan_s: 33 ints
// of shared memory.  Ends with a barrier (sel is ready to read).
__device__ __forceinline__ void block_topc_mark(const uint32_t* key, int n, int C, uint8_t* sel, int* hist, int* scan_s) {
  const int tid = threadIdx.x, nth = blockDim.x, lane = tid & 31;
  if (C >= n || C <= 0) {
    for (int i = tid; i < n; i += nth) sel[i] = C >= n ? 1 : 0;
    __syncthreads();
    return;
  }
  uint32_t prefix = 0u, mask = 0u;
  int need = C;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += nth) hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += nth) {
      const uint32_t k = key[i];
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid < 32) {
      // digits from the largest down: the first one whose cumulative count reaches `need`
      int run = 0, found = -1, above = 0;
      for (int base = 255; base >= 0 && found < 0; base -= 32) {
        const int c = hist[base - lane];                // lane 0 holds the largest digit of this group of 32
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
      if (lane == 0) { hist[256] = found; hist[257] = above; }
    }
    __syncthreads();
    prefix |= (uint32_t)hist[256] << shift;
    mask |= 0xFFu << shift;
    need -= hist[257];
    __syncthreads();
  }
  // prefix = T; need = how many keys equal to T are taken, lowest index first
  int eq_base = 0;
  for (int c0 = 0; c0 < n; c0 += nth) {
    const int i = c0 + tid;
    const uint32_t k = i < n ? key[i] : 0u;
    const int eq = (i < n && k == prefix) ? 1 : 0;
    int tot;
    const int pre = block_excl_scan(eq, scan_s, tot);
    if (i < n) sel[i] = (k > prefix || (eq && eq_base + pre < need)) ? 1 : 0;
    eq_base += tot;
  }
  __syncthreads();
}

struct AttnArgs {
  focus_shape sh;
  float scale;
  const void* Q;
  int q_base, n_q;
  const int32_t* q_rows;
  const int32_t* n_rows;
  int max_rows;       // host bound on rows (n_q when q_rows == NULL)
  const void* K;
  const void* V;
  int dense;          // 1: key set = [0, L)
  int group_stride;   // block list row of KV head g = g * group_stride (1 per-group lists, 0 shared list)
  const int32_t* block_idx;
  int max_blocks;
  const int32_t* block_cnt;
  const int32_t* sink_idx;
  const uint8_t* sink_keep;
  int n_sink;
  void* O;            // may be NULL (lse only)
  float* lse;         // may be NULL
  int lse_stride;
};

struct SinkGather {          // sink rows of one layer gathered into compact per-KV-head tiles
  __nv_bfloat16* gK;         // [Hkv][ns_pad][128]
  __nv_bfloat16* gV;
  uint8_t* mask;             // [Hkv][ns_pad]: 1 = attend this column
};

focus_status launch_attn_simt(focus_ctx* ctx, const AttnArgs& a, cudaStream_t st);
focus_status launch_attn_tc_ws(focus_ctx* ctx, const AttnArgs& a, WsAlloc& ws, const SinkGather* pre, cudaStream_t st);
focus_status launch_attn_tc(focus_ctx* ctx, const AttnArgs& a, cudaStream_t st);
bool attn_tc_supported(const focus_ctx* ctx, const AttnArgs& a);
size_t attn_tc_workspace(const focus_shape* s, int n_q, int max_blocks, int n_sink);
