// Internal declarations shared by the translation units of libh2o_b200.so.
// Nothing here is part of the public ABI (see include/h2o.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "h2o.h"

struct CUtensorMap_st;  // <cuda.h>

namespace h2o {

// Static description of one unit, stored in launch order (largest budget first).
struct UnitMeta {
  int64_t slot_off;  // first slot of the unit (a multiple of 4)
  int32_t unit;      // sequence * n_heads + head
  int32_t kbud;      // heavy budget k
  int32_t rwin;      // recent window r
  int32_t pad_;
};

// Device-side view of a cache.  All pointers live inside the caller's workspace.
// `meta`, `count` and `tpos` are indexed by launch position, not by unit.
struct CacheView {
  void* K;               // [total_slots][d] storage dtype
  void* V;               // [total_slots][d]
  double* acc;           // [total_slots] accumulated attention score
  int32_t* pos;          // [total_slots] token position held by the slot
  int32_t* count;        // [units] occupied slots
  int32_t* tpos;         // [units] position of the next token
  int32_t* status;       // [1] first error recorded by a kernel
  const UnitMeta* meta;  // [units]
  int32_t units, n_heads, head_dim;
  float scale;           // softmax scale c
  // When every sequence has the same budgets the unit table is arithmetic (unit = launch position,
  // slot_off = position * uni_pad) and a block need not load it: uni_pad = slots per unit rounded up
  // to 4, uni_k / uni_r the budgets; uni_pad < 0 otherwise.
  int32_t uni_pad, uni_k, uni_r;
  // 0: candidates are ranked by the accumulated score (Algorithm 2); 1: by the averaged score, accumulated
  // score / number of queries that attended the key ("Discussions and Limitations").  Stored scores are the
  // accumulated ones in both modes.
  int32_t score_mode;
  int32_t kv4;  // 1: K/V slots are 80-byte 4-bit rows (written by the kernels of decode_kv4.cu)
  // Sparse pattern inside the recent window (heavy hitters combined with the strided / fixed Sparse Transformer
  // patterns, Section 5.1): 0 none, 1 strided(stride mask_a, local window mask_b), 2 fixed(block mask_a, mask_b
  // summary columns).  See key_attended().
  int32_t mask_kind, mask_a, mask_b;
  // "Top-K" attention in decode steps (appendix "Enhancing the Top-K baseline"): > 0: a query attends only its topk
  // largest logits among what it would otherwise attend (equal logits: the higher position); 0: off.
  int32_t topk;
  const int32_t* seq_rwin;  // [batch] recent window of every sequence (the prompt kernels index by unit, not by launch position)
  int64_t total_slots;      // slots of all units together (the limit of every slot index)
  int32_t group;            // query heads per unit (grouped-query attention); 1: every head has its own cache
};

// Debug build (-DH2O_BOUNDS, the stand-in for a memory checker): every slot, unit and prompt-row index that
// addresses the cache, the prompt tensors or the per-unit arrays is checked right before it is used; a violation
// records H2O_ERR_STATE in the cache's status word and the access is skipped.  In normal builds the checks
// compile to nothing.
#ifdef H2O_BOUNDS
__device__ __forceinline__ bool index_in_range(long long idx, long long limit, int32_t* status) {
  if (idx >= 0 && idx < limit) return true;
  atomicCAS(status, 0, H2O_ERR_STATE);
  return false;
}
#define H2O_IN_RANGE(idx, limit, status) ::h2o::index_in_range((long long)(idx), (long long)(limit), (status))
#else
#define H2O_IN_RANGE(idx, limit, status) true
#endif

// Does the query at position t attend the key at position p (r = the unit's recent window)?  The token itself and
// everything older than the window (heavy hitters, and the entry that has just left the window) always; of the
// window what the pattern allows.
__device__ __forceinline__ bool key_attended(int kind, int a, int b, int p, int t, int r) {
  if (kind == 0 || p == t || p <= t - r) return true;
  if (kind == 1) return (t - p) < b || (t - p) % a == 0;
  return p / a == t / a || p % a >= a - b;
}

// Scratch of one prefill call; per-head planes so that a unit's rows are contiguous:
// index = h * total_tokens + token (row statistics: h = QUERY head, n_heads * group planes; column sums: K/V head).
struct PrefillScratch {
  float* rowmax;   // m_i
  float* rowsum;   // l_i
  float2* rowstat; // tensor-core path: {reference maximum (log2 domain), 1 / row sum}; aliases rowmax/rowsum
  double* acc0;    // column sums
  int32_t* cu;     // [batch + 1] device copy of cu_seqlens
  int32_t* work;   // two work counters of the persistent prefill kernels, zero when the launch starts
  // item order of the persistent forward kernel (host-built): first item index of every group of units
  const int32_t* item_base;  // [fs_groups + 1]
  int32_t fs_grp, fs_groups, fs_items;
  int64_t total_tokens;
};

// Read-only view of a handle's configuration (budget arrays are the handle's own copies).
const h2o_config_t* cache_config(const h2o_cache_t* cache);

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) is a per-device setting: remember per kernel and
// device whether it has been raised already.  `flags` is a zero-initialised static of the caller.
inline cudaError_t ensure_dynamic_smem(const void* func, int bytes, unsigned long long* flags) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (*flags & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) *flags |= bit;
  return e;
}

// SMs of the current device (asked once per device; the dispatch thresholds of the launchers scale with it).
inline int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

// Launchers (each returns the cudaError_t of its launch).
// `split` thread blocks (one cluster) share a unit, each owning `chunk` consecutive slots.
// `stages` is the depth of the shared-memory ring (0 = default).  `quiescent`: nothing this library
// launched immediately before on the stream can have written this cache, so the kernel may read the
// cache before the previous kernel of the stream has finished (it still waits before reading q/k/v).
// `all_full`: the host knows that every unit holds exactly its budget of entries, so blocks need not
// load the counters before they start streaming.
cudaError_t launch_decode(const CacheView& c, int dtype, int split, int chunk, int stages, bool quiescent, bool all_full,
                          const void* q, const void* k_new, const void* v_new, void* out, int32_t* evicted_pos,
                          cudaStream_t stream);
// Grouped-query attention (c.group query heads per unit): one block per unit, K and V rows read once for the group.
size_t decode_gqa_smem_bytes(int group, int max_B, int head_dim);
cudaError_t launch_decode_gqa(const CacheView& c, int dtype, int max_B, bool cache_is_quiescent, bool all_full, const void* q,
                              const void* k_new, const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream);
// The streaming form for bf16 / head_dim 128 (decode_two_pass.cu); launch_decode_gqa uses it when it is supported.
bool decode_two_pass_supported(int dtype, int head_dim, int group, int chunk);
cudaError_t launch_decode_two_pass(const CacheView& c, int split, int chunk, bool cache_is_quiescent, bool all_full,
                                   const void* q, const void* k_new, const void* v_new, void* out, int32_t* evicted_pos,
                                   cudaStream_t stream);
// ALU path; `rows` = attention rows + row statistics, `colsum` = column sums.
cudaError_t launch_prefill_naive(const CacheView& c, const PrefillScratch& s, int dtype, int max_seqlen, const void* q,
                                 const void* k, const void* v, void* out, bool rows, bool colsum, cudaStream_t stream);
// Tensor-core path (bf16, head_dim 128 only).
bool prefill_tc_supported(int dtype, int head_dim);
cudaError_t launch_fwd_tc(const CacheView& c, const PrefillScratch& s, int max_seqlen, const void* q, const void* k,
                          const void* v, void* out, cudaStream_t stream);
cudaError_t launch_colsum_tc(const CacheView& c, const PrefillScratch& s, int max_seqlen, const void* q, const void* k,
                             cudaStream_t stream);
// Tensor map over a [rows][n_heads][128] bf16 array: box = box_rows x 1 head x 64 elements, 128-byte swizzle.
bool make_tile_map(CUtensorMap_st* map, const void* base, int64_t rows, int n_heads, int box_rows);
// Up to kDecodeChunkTokens consecutive decode steps per launch (bf16, head_dim 128, small budgets);
// inputs and outputs are [n_tokens][units][head_dim], evicted_pos [n_tokens][units] (nullable).
constexpr int kDecodeChunkTokens = 32;
bool decode_chunk_supported(int dtype, int head_dim, int max_B, int64_t total_slots);
cudaError_t launch_fscore(const CacheView& c, int hkind, double* out, cudaStream_t stream);
size_t kv4_row_bytes();
int fwd_group_units(int units, int max_seqlen);
cudaError_t launch_decode_kv4(const CacheView& c, int split, int chunk, bool cache_is_quiescent, bool all_full, const void* q,
                              const void* k_new, const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream);
cudaError_t launch_gather_kv4(const CacheView& c, const PrefillScratch& s, const void* k, const void* v, cudaStream_t stream);
// `meta`: host copy of the unit table in launch order.
cudaError_t launch_decode_chunk(const CacheView& c, int64_t total_slots, const UnitMeta* meta, const void* q,
                                const void* k, const void* v, int n_tokens, void* out, int32_t* evicted_pos,
                                cudaStream_t stream);
// One warp waits `polls` times on a barrier nobody arrives at, then records H2O_ERR_TIMEOUT (diagnostic).
cudaError_t launch_wait_probe(const CacheView& c, uint32_t polls, cudaStream_t stream);
cudaError_t launch_select_gather(const CacheView& c, const PrefillScratch& s, int dtype, int max_B, int max_seqlen, const void* k,
                                 const void* v, cudaStream_t stream);

// ---------------------------------------------------------------------------
// Small device helpers
// ---------------------------------------------------------------------------
template <typename T>
struct Vec16;  // 16-byte vector of T, widened to float on load

template <>
struct Vec16<float> {
  static constexpr int N = 4;
  __device__ __forceinline__ static void load(const float* p, float (&f)[4]) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ __forceinline__ static void store(float* p, const float (&f)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
  }
};

template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ __forceinline__ static void unpack(const uint4& v, float (&f)[8]) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
  }
  __device__ __forceinline__ static void load(const __nv_bfloat16* p, float (&f)[8]) {
    unpack(*reinterpret_cast<const uint4*>(p), f);
  }
  __device__ __forceinline__ static uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&b);
  }
  __device__ __forceinline__ static void store(__nv_bfloat16* p, const float (&f)[8]) {
    uint4 v;
    v.x = pack2(f[0], f[1]); v.y = pack2(f[2], f[3]); v.z = pack2(f[4], f[5]); v.w = pack2(f[6], f[7]);
    *reinterpret_cast<uint4*>(p) = v;
  }
};

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

}  // namespace h2o
