// Several consecutive decode steps in one launch (bf16, head_dim 128, budget + 32 <= 512 slots).
//
// Algorithm 1 of the paper runs token by token: token i attends over S_{i-1} and itself, the scores
// are accumulated, one entry is evicted.  Each eviction depends on every earlier row, so the steps
// cannot run in parallel — but the raw dot products can: q_i . k_x does not depend on which entries
// are still alive.  For a chunk of up to 32 tokens this kernel therefore
//   1. computes S^T = K Q^T for ALL keys in play (the cached entries and the chunk's own keys) on
//      the tensor cores, accumulators in tensor memory: one TMEM lane = one key, one column = one
//      token of the chunk;
//   2. walks the tokens in order with ONE THREAD PER KEY holding that key's scores, its accumulated
//      score (fp64), position, slot and an alive flag in registers: softmax over the live set, score
//      accumulation, eviction of the minimum under (score, position) — two block-wide reductions per
//      token, no global memory traffic;
//   3. writes the probabilities (bf16 hi + lo, zero for dead or unborn keys) to shared memory and
//      computes O^T = V^T P^T on the tensor cores;
//   4. writes the surviving chunk entries into the slots they inherited from their victims.
// The result equals that of the same number of single decode steps (same set semantics, same order).
//
// Paper: Algorithm 1 / Algorithm 2 (token-by-token eviction), Section 4.2 (greedy eviction policy).
#include <climits>

#include "h2o_internal.cuh"
#include "sm100_ptx.cuh"

namespace h2o {

namespace {

using namespace ptx;

constexpr int kD = 128;
constexpr int kC = kDecodeChunkTokens;      // tokens per launch
constexpr int kKeyThreads = 512;            // one thread per key row
constexpr int kKeyWarps = kKeyThreads / 32;
constexpr int kThreads = kKeyThreads + 32;  // + control warp (TMA and MMA issue)
constexpr int kTileRows = 128;
constexpr int kHalfBytes = kTileRows * 128;  // 128 rows x 64 bf16
constexpr int kTileBytes = 2 * kHalfBytes;   // two halves cover head_dim 128
constexpr int kMaxTiles = kKeyThreads / kTileRows;
constexpr int kQHalfBytes = kC * 128;
constexpr int kPBlockBytes = kC * 128;               // 64 keys x kC tokens of bf16
constexpr int kPBufBytes = (kKeyThreads / 64) * kPBlockBytes;
constexpr int kTmemCols = 256;
constexpr uint32_t kColS = 0;    // S^T of key tile m: columns [m * kC, (m + 1) * kC)
constexpr uint32_t kColO = 128;  // O^T: kC columns
constexpr int kDynSmem = kMaxTiles * kTileBytes + 2 * kPBufBytes + 2 * kQHalfBytes + 1024;
static_assert(kMaxTiles * kC <= (int)kColO && kColO + kC <= kTmemCols, "tensor memory columns");

struct KeyCand {
  unsigned long long key;  // bit pattern of the accumulated score (>= 0, so it orders like the value)
  int pos;
  int slot;
  int x;  // key index inside the block; -1: none
  int pad_;
};

struct Shared {
  uint64_t k_full, k_ready, s_full, v_full, p_ready, o_full;
  uint32_t tmem_base;
  int abort_flag;
  float wmax[kKeyWarps][kC];
  float m_row[kC];
  float red_sum[2][kKeyWarps];
  float red_max[kKeyWarps];
  KeyCand red_cand[2][kKeyWarps];
  int evicted[kC];
  int wb_slot[kC];
};

// Optional cycle stamps of block 0 (compile with -DH2O_PHASE_TIMERS).
#ifdef H2O_PHASE_TIMERS
__device__ long long g_chunk_prof[16];
#define DC_STAMP(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) g_chunk_prof[i] = clock64(); } while (0)
#else
#define DC_STAMP(i) do { } while (0)
#endif

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void key_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kKeyThreads) : "memory"); }

// Byte offset of 16-byte piece `c16` (0..7) of row `row` inside a 128-byte-swizzled block of 128-byte rows.
__device__ __forceinline__ uint32_t swz(int row, int c16) {
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((c16 ^ (row & 7)) << 4));
}

// Sum over the 16 per-warp values held by lanes 0..15 (and mirrored in 16..31); same order in every warp.
__device__ __forceinline__ float sum16(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 8);
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v;
}

// Warp-wide minimum under (score, position); every lane gets the winner.
__device__ __forceinline__ KeyCand warp_argmin(const KeyCand& a) {
  const bool valid = a.x >= 0;
  const unsigned long long bits = valid ? a.key : ~0ull;
  const unsigned hi = (unsigned)(bits >> 32), lo = (unsigned)bits;
  const unsigned mh = __reduce_min_sync(0xffffffffu, hi);
  const unsigned ml = __reduce_min_sync(0xffffffffu, hi == mh ? lo : 0xffffffffu);
  const bool tie = valid && hi == mh && lo == ml;
  const unsigned mp = __reduce_min_sync(0xffffffffu, tie ? (unsigned)a.pos : 0xffffffffu);
  const unsigned who = __ballot_sync(0xffffffffu, tie && (unsigned)a.pos == mp);
  KeyCand b;
  b.key = ((unsigned long long)mh << 32) | ml;
  b.pos = (int)mp;
  b.pad_ = 0;
  if (who == 0) {
    b.slot = -1;
    b.x = -1;
    return b;
  }
  const int src = __ffs(who) - 1;
  b.slot = __shfl_sync(0xffffffffu, a.slot, src);
  b.x = __shfl_sync(0xffffffffu, a.x, src);
  return b;
}

__global__ void __launch_bounds__(kThreads, 1)
decode_chunk_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, CacheView c, const __nv_bfloat16* __restrict__ k_in,
                    const __nv_bfloat16* __restrict__ v_in, __nv_bfloat16* __restrict__ out,
                    int32_t* __restrict__ evicted_pos, int tok0, int n_tok) {
  extern __shared__ unsigned char dyn_raw[];
  __shared__ Shared sh;
  unsigned char* dyn = dyn_raw + ((1024u - (smem_u32(dyn_raw) & 1023u)) & 1023u);
  unsigned char* kv = dyn;                                   // key tiles, later value tiles
  unsigned char* p_hi = dyn + kMaxTiles * kTileBytes;        // [8 blocks of 64 keys][kC tokens][128 B]
  unsigned char* p_lo = p_hi + kPBufBytes;
  unsigned char* q_s = p_lo + kPBufBytes;                    // [2 halves][kC tokens][128 B]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int su = blockIdx.x;
  const UnitMeta mt = c.meta[su];
  const int u = mt.unit, r = mt.rwin, B = mt.kbud + mt.rwin;
  const int cnt0 = c.count[su], t0 = c.tpos[su];
  const int ceff = min(kC, n_tok - tok0);
  const int nk = cnt0 + ceff;                          // keys in play: cached entries, then the chunk's own
  const int ntiles = (nk + kTileRows - 1) / kTileRows;
  if (nk > kKeyThreads || ceff < 1) {                  // the host never launches this; leave before any barrier exists
    if (tid == 0) atomicCAS(c.status, 0, H2O_ERR_STATE);
    return;
  }
  const int64_t in_stride = (int64_t)c.units * kD;     // elements between consecutive tokens of the inputs
  const __nv_bfloat16* k_u = k_in + ((int64_t)tok0 * c.units + u) * kD;
  const __nv_bfloat16* v_u = v_in + ((int64_t)tok0 * c.units + u) * kD;

  if (tid == 0) {
    mbar_init(&sh.k_full, 1);
    mbar_init(&sh.k_ready, kKeyThreads);
    mbar_init(&sh.s_full, 1);
    mbar_init(&sh.v_full, 1);
    mbar_init(&sh.p_ready, kKeyThreads);
    mbar_init(&sh.o_full, 1);
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kKeyWarps) tmem_alloc(&sh.tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;

  if (warp == kKeyWarps) {
    // ---------------- control warp: loads and matrix instructions ----------------
    bool ok = true;
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      mbar_expect_tx(&sh.k_full, (uint32_t)(ntiles * kTileBytes + 2 * kQHalfBytes));
      tma_load_3d(q_s, &map_q, 0, u, tok0, &sh.k_full);
      tma_load_3d(q_s + kQHalfBytes, &map_q, 64, u, tok0, &sh.k_full);
      for (int m = 0; m < ntiles; ++m) {
        const int row = (int)mt.slot_off + m * kTileRows;
        tma_load_3d(kv + m * kTileBytes, &map_k, 0, 0, row, &sh.k_full);
        tma_load_3d(kv + m * kTileBytes + kHalfBytes, &map_k, 64, 0, row, &sh.k_full);
      }
    }
    // S^T = K Q^T once the key threads have put the chunk's own keys behind the cached ones
    ok = wait_or_abort(&sh.k_ready, 0, abort_flag);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    if (ok && elect_one()) {
      constexpr uint32_t idesc_s = instr_desc_f16(kTileRows, kC, kFmtBF16, kFmtBF16, false, false);
      const uint32_t a0 = smem_u32(kv), b0 = smem_u32(q_s);
      for (int m = 0; m < ntiles; ++m) {
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t offa = (uint32_t)m * kTileBytes + (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
          const uint32_t offb = (uint32_t)(ks >> 2) * kQHalfBytes + (uint32_t)(ks & 3) * 32u;
          mma_ss(tmem + kColS + (uint32_t)(m * kC), smem_desc_sw128(a0 + offa, 16, 1024),
                 smem_desc_sw128(b0 + offb, 16, 1024), idesc_s, ks > 0);
        }
      }
      mma_commit(&sh.s_full);
    }
    __syncwarp();
    // the key tiles are dead once the scores exist: the values take their place
    ok = ok && wait_or_abort(&sh.s_full, 0, abort_flag);
    ok = __all_sync(0xffffffffu, ok);
    if (ok && lane == 0) {
      mbar_expect_tx(&sh.v_full, (uint32_t)(ntiles * kTileBytes));
      for (int m = 0; m < ntiles; ++m) {
        const int row = (int)mt.slot_off + m * kTileRows;
        tma_load_3d(kv + m * kTileBytes, &map_v, 0, 0, row, &sh.v_full);
        tma_load_3d(kv + m * kTileBytes + kHalfBytes, &map_v, 64, 0, row, &sh.v_full);
      }
    }
    __syncwarp();
    // O^T = V^T P^T (hi and lo halves of P) once every token's probabilities are in shared memory
    ok = ok && wait_or_abort(&sh.p_ready, 0, abort_flag);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    if (ok && elect_one()) {
      constexpr uint32_t idesc_o = instr_desc_f16(kD, kC, kFmtBF16, kFmtBF16, true, false);
      const uint32_t v0 = smem_u32(kv), ph = smem_u32(p_hi), pl = smem_u32(p_lo);
      bool first = true;
      for (int kb = 0; kb < 2 * ntiles; ++kb) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint32_t offv = (uint32_t)(kb >> 1) * kTileBytes + (uint32_t)(((kb & 1) * 64 + ks * 16) * 128);
          const uint32_t offp = (uint32_t)kb * kPBlockBytes + (uint32_t)ks * 32u;
          const uint64_t da = smem_desc_sw128(v0 + offv, kHalfBytes, 1024);
          mma_ss(tmem + kColO, da, smem_desc_sw128(ph + offp, 16, 1024), idesc_o, !first);
          mma_ss(tmem + kColO, da, smem_desc_sw128(pl + offp, 16, 1024), idesc_o, true);
          first = false;
        }
      }
      mma_commit(&sh.o_full);
    }
    __syncwarp();
  } else {
    // ---------------- key threads ----------------
    const int x = tid;  // key index: tile x / 128, TMEM lane x % 128
    bool ok = true;
    bool alive = x < cnt0;
    double acc = 0.0;
    int pos = 0, slot = x;
    if (alive) {
      acc = c.acc[mt.slot_off + x];
      pos = c.pos[mt.slot_off + x];
    }
    // the chunk's own key rows go behind the cached ones (row cnt0 + j), in the layout the TMA wrote
    DC_STAMP(0);
    ok = wait_or_abort(&sh.k_full, 0, abort_flag);
    DC_STAMP(1);
    {
      const int j = tid >> 4, c16 = tid & 15;
      if (j < ceff) {
        const uint4 val = *reinterpret_cast<const uint4*>(k_u + (int64_t)j * in_stride + c16 * 8);
        const int row = cnt0 + j;
        unsigned char* dst = kv + (row >> 7) * kTileBytes + (c16 >> 3) * kHalfBytes + swz(row & 127, c16 & 7);
        *reinterpret_cast<uint4*>(dst) = val;
      }
    }
    fence_proxy_async();
    mbar_arrive(&sh.k_ready);

    // this key's raw scores against the chunk's tokens
    float s[kC];
#pragma unroll
    for (int i = 0; i < kC; ++i) s[i] = 0.f;
    ok = wait_or_abort(&sh.s_full, 0, abort_flag) && ok;
    ok = __all_sync(0xffffffffu, ok);
    DC_STAMP(2);
    tc_fence_after();
    if (ok && (warp >> 2) < ntiles) {
      uint32_t raw[32];
      tmem_ld32(tmem + kColS + (uint32_t)((warp >> 2) * kC) + ((uint32_t)((warp & 3) * 32) << 16), raw);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < kC; ++i) s[i] = c.scale * __uint_as_float(raw[i]);
    }
    // reference maximum of every token's row: over all keys that exist at that token (alive or not;
    // any reference works for a softmax, and this one needs no reduction inside the sequential loop)
    const int jx = x - cnt0;  // index of this key inside the chunk (if >= 0)
    {
      float mine = -INFINITY;
#pragma unroll
      for (int i = 0; i < kC; ++i) {
        const bool valid = x < cnt0 || (jx < ceff && jx <= i);
        const float v = warp_max(valid ? s[i] : -INFINITY);
        if (lane == i) mine = v;
      }
      sh.wmax[warp][lane] = mine;
      key_sync();
      if (tid < kC) {
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < kKeyWarps; ++w) m = fmaxf(m, sh.wmax[w][tid]);
        sh.m_row[tid] = m;
      }
      key_sync();
    }

    DC_STAMP(3);
    // ---- the tokens, in order (Algorithm 1) ----
    int live = cnt0;  // entries in the cache before the current token
    const uint32_t pcol = (uint32_t)((x >> 6) * kPBlockBytes + (x & 7) * 2);
    const int pc16 = (x & 63) >> 3;
#pragma unroll
    for (int i = 0; i < kC; ++i) {
      if (i < ceff) {
        const int t = t0 + i;
        const bool is_new = jx == i;
        if (is_new) {  // the token's own key enters the set with an empty score
          alive = true;
          acc = 0.0;
          pos = t;
          slot = -1;
        }
        float e = alive ? expf(s[i] - sh.m_row[i]) : 0.f;
        {
          const float ws = warp_sum(e);
          if (lane == 0) sh.red_sum[i & 1][warp] = ws;
        }
        key_sync();
        float l = sum16(sh.red_sum[i & 1][lane & 15]);
        if (!(l > 1e-30f)) {  // every live score sits far below a dead key's: use the live maximum instead
          const float wm = warp_max(alive ? s[i] : -INFINITY);
          if (lane == 0) sh.red_max[warp] = wm;
          key_sync();
          float m = sh.red_max[lane & 15];
          m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
          m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
          m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
          m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
          e = alive ? expf(s[i] - m) : 0.f;
          const float ws = warp_sum(e);
          key_sync();  // everyone has read red_sum and red_max
          if (lane == 0) sh.red_sum[i & 1][warp] = ws;
          key_sync();
          l = sum16(sh.red_sum[i & 1][lane & 15]);
        }
        const float p = e / l;
        if (alive) acc += (double)p;  // Algorithm 2: accumulated score
        {
          const __nv_bfloat16 hi = __float2bfloat16_rn(p);
          const __nv_bfloat16 lo = __float2bfloat16_rn(p - __bfloat162float(hi));
          const uint32_t off = pcol + (uint32_t)((i >> 3) * 1024 + (i & 7) * 128 + ((pc16 ^ (i & 7)) << 4));
          *reinterpret_cast<__nv_bfloat16*>(p_hi + off) = hi;
          *reinterpret_cast<__nv_bfloat16*>(p_lo + off) = lo;
        }
        if (live >= B) {  // full: evict the minimum among the entries outside the recent window
          KeyCand cd;
          cd.key = (unsigned long long)__double_as_longlong(acc);
          cd.pos = pos;
          cd.slot = slot;
          cd.x = (alive && pos <= t - r) ? x : -1;
          cd.pad_ = 0;
          const KeyCand wb = warp_argmin(cd);
          if (lane == 0) sh.red_cand[i & 1][warp] = wb;
          key_sync();
          const KeyCand vic = warp_argmin(sh.red_cand[i & 1][lane & 15]);
          if (vic.x >= 0) {
            if (x == vic.x) alive = false;
            else if (is_new) slot = vic.slot;  // in-place replacement of the victim
            if (tid == 0) sh.evicted[i] = vic.pos;
          } else {  // a full cache always has a candidate; record instead of corrupting
            if (is_new) alive = false;
            if (tid == 0) {
              sh.evicted[i] = -1;
              atomicCAS(c.status, 0, H2O_ERR_STATE);
            }
          }
        } else {
          if (is_new) slot = live;
          live += 1;
          if (tid == 0) sh.evicted[i] = -1;
        }
      }
    }

    // ---- values: the chunk's own rows behind the cached ones, zeros in the rows no key owns ----
    DC_STAMP(4);
    ok = wait_or_abort(&sh.v_full, 0, abort_flag) && ok;
    DC_STAMP(5);
    {
      const int j = tid >> 4, c16 = tid & 15;
      if (j < ceff) {
        const uint4 val = *reinterpret_cast<const uint4*>(v_u + (int64_t)j * in_stride + c16 * 8);
        const int row = cnt0 + j;
        unsigned char* dst = kv + (row >> 7) * kTileBytes + (c16 >> 3) * kHalfBytes + swz(row & 127, c16 & 7);
        *reinterpret_cast<uint4*>(dst) = val;
      }
      const int nzero = (ntiles * kTileRows - nk) * 16;
      for (int idx = tid; idx < nzero; idx += kKeyThreads) {
        const int row = nk + (idx >> 4), z16 = idx & 15;
        unsigned char* dst = kv + (row >> 7) * kTileBytes + (z16 >> 3) * kHalfBytes + swz(row & 127, z16 & 7);
        *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    fence_proxy_async();
    mbar_arrive(&sh.p_ready);

    DC_STAMP(6);
    // ---- write the state back: scores of the survivors, the chunk's surviving rows into their slots ----
    if (alive) {
      c.acc[mt.slot_off + slot] = acc;
      if (jx >= 0) c.pos[mt.slot_off + slot] = pos;
    }
    if (jx >= 0 && jx < ceff) sh.wb_slot[jx] = alive ? slot : -1;
    key_sync();
    for (int idx = tid; idx < ceff * 32; idx += kKeyThreads) {
      const int j = idx >> 5, pc = idx & 31, c16 = pc & 15;
      const int sl = sh.wb_slot[j];
      if (sl >= 0) {
        const __nv_bfloat16* src = (pc < 16 ? k_u : v_u) + (int64_t)j * in_stride + c16 * 8;
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(pc < 16 ? c.K : c.V) + (mt.slot_off + sl) * kD + c16 * 8;
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
      }
    }
    if (tid == 0) {
      c.count[su] = live;
      c.tpos[su] = t0 + ceff;
    }
    if (tid < ceff && evicted_pos) evicted_pos[(int64_t)(tok0 + tid) * c.units + u] = sh.evicted[tid];

    // ---- outputs: lane = head dimension, column = token ----
    DC_STAMP(7);
    if (warp < 4) {
      ok = wait_or_abort(&sh.o_full, 0, abort_flag) && ok;
      DC_STAMP(8);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      if (ok) {
        uint32_t o[32];
        tmem_ld32(tmem + kColO + ((uint32_t)(warp * 32) << 16), o);
        tmem_wait_ld();
        __nv_bfloat16* out_u = out + ((int64_t)tok0 * c.units + u) * kD + tid;
#pragma unroll
        for (int i = 0; i < kC; ++i)
          if (i < ceff) out_u[(int64_t)i * in_stride] = __float2bfloat16_rn(__uint_as_float(o[i]));
      }
    }
  }
  DC_STAMP(9);
  tc_fence_before();
  __syncthreads();
  DC_STAMP(10);
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
  if (warp == kKeyWarps) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace

#ifdef H2O_PHASE_TIMERS
extern "C" int h2o_debug_chunk_prof(long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_chunk_prof, sizeof(long long) * 16);
}
#endif

bool decode_chunk_supported(int dtype, int head_dim, int max_B, int64_t total_slots) {
  return prefill_tc_supported(dtype, head_dim) && max_B + kC <= kKeyThreads && total_slots < INT_MAX - kTileRows;
}

cudaError_t launch_decode_chunk(const CacheView& c, int64_t total_slots, const void* q, const void* k, const void* v,
                                int n_tokens, void* out, int32_t* evicted_pos, cudaStream_t stream) {
  CUtensorMap map_q, map_k, map_v;
  if (!make_tile_map(&map_q, q, n_tokens, c.units, kC) || !make_tile_map(&map_k, c.K, total_slots, 1, kTileRows) ||
      !make_tile_map(&map_v, c.V, total_slots, 1, kTileRows))
    return cudaErrorInvalidValue;
  static unsigned long long attr_flags = 0;
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_chunk_kernel), kDynSmem, &attr_flags);
    if (e != cudaSuccess) return e;
  }
  for (int tok0 = 0; tok0 < n_tokens; tok0 += kC) {
    decode_chunk_kernel<<<(unsigned)c.units, kThreads, kDynSmem, stream>>>(
        map_q, map_k, map_v, c, static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v),
        static_cast<__nv_bfloat16*>(out), evicted_pos, tok0, n_tokens);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace h2o
