// Several consecutive decode steps in one launch (bf16, head_dim 128, budget + 32 <= 1024 slots).
//
// Algorithm 1 of the paper runs token by token: token i attends over S_{i-1} and itself, the scores
// are accumulated, one entry is evicted.  Each eviction depends on every earlier row, so the steps
// cannot run in parallel — but the raw dot products can: q_i . k_x does not depend on which entries
// are still alive.  For a chunk of up to 32 tokens this kernel therefore
//   1. computes S^T = K Q^T for ALL keys in play (the cached entries and the chunk's own keys) on
//      the tensor cores, accumulators in tensor memory: one TMEM lane = one key, one column = one
//      token of the chunk;
//   2. turns them into exponentials relative to a per-token reference maximum (any reference gives
//      the same softmax), all tokens at once;
//   3. walks the tokens in order.  Four warps; a thread owns up to 2, 4 or 8 keys (one per 128-key tile:
//      a warp can only read its own quarter of the TMEM lanes) with their exponentials, accumulated
//      scores (fp64), positions, slots and alive flags in registers.  Per token ONE exchange between
//      the warps carries both the eviction candidates of this token and the partial sums of the next
//      token's normaliser (taken over the set before the eviction; the victim's own term is then
//      subtracted, or the sum redone if that term is large enough for cancellation to matter);
//   4. writes the probabilities (bf16 hi + lo, zero for dead or unborn keys) to shared memory and
//      computes O^T = V^T P^T on the tensor cores;
//   5. writes the surviving chunk entries into the slots they inherited from their victims.
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
constexpr int kKeyWarps = 4;                // one per quarter of the TMEM lanes
constexpr int kKeyThreads = kKeyWarps * 32;
constexpr int kThreads = kKeyThreads + 32;  // + control warp (TMA and MMA issue)
constexpr int kTileRows = 128;
constexpr int kMaxTiles = 8;                // most keys per thread (the kernel is compiled for 2, 4 and 8)
constexpr int kMaxKeys = kMaxTiles * kTileRows;
constexpr int kMaxBatches = 4;
// key / value tiles resident in shared memory at a time, by keys per thread
__host__ __device__ constexpr int batch_tiles(int kt) { return kt <= 2 ? 1 : 2; }
constexpr int kHalfBytes = kTileRows * 128;  // 128 rows x 64 bf16
constexpr int kTileBytes = 2 * kHalfBytes;   // two halves cover head_dim 128
constexpr int kQHalfBytes = kC * 128;
constexpr int kPBlockBytes = kC * 128;       // 64 keys x kC tokens of bf16
constexpr uint32_t kColS = 0;                // key tile m: columns [m * kC, (m + 1) * kC); O^T behind the last tile

// Shared memory holds one batch of tiles (keys first, values later), the probabilities of that batch
// as bf16 hi and lo, and the chunk's queries; tensor memory is sized by the tiles of the largest unit.
__host__ __device__ constexpr int dyn_smem_bytes(int kt) {
  return batch_tiles(kt) * (kTileBytes + 4 * kPBlockBytes) + 2 * kQHalfBytes + 1024;
}
__host__ __device__ constexpr uint32_t tmem_cols(int tiles) {
  return tiles <= 1 ? 64u : tiles <= 3 ? 128u : tiles <= 7 ? 256u : 512u;
}

struct Shared {
  uint64_t k_full[kMaxBatches], k_ready[kMaxBatches], s_done[kMaxBatches];
  uint64_t v_full[kMaxBatches], p_ready[kMaxBatches], o_done[kMaxBatches];
  uint32_t tmem_base;
  int abort_flag;
  float wmax[kKeyWarps][kC];
  float m_row[kC];
  // what each warp posts per token (two buffers, by token parity): its eviction candidate for this
  // token and its share of the next token's normaliser
  __align__(16) unsigned long long post_key[2][kKeyWarps];  // bit pattern of the candidate's score (>= 0: orders like the value); ~0: none
  __align__(16) int post_pos[2][kKeyWarps];                 // INT_MAX: none
  __align__(16) float post_sum[2][kKeyWarps];               // next row's exponentials over the warp's live keys (before the eviction)
  int post_slot[2][kKeyWarps];
  int post_x[2][kKeyWarps];       // candidate's key index inside the block; -1: none
  float post_enext[2][kKeyWarps]; // the candidate's exponential in the next row
  float redo[kKeyWarps], redo2[kKeyWarps];
  int evicted[kC];
  int wb_slot[kC];
};

// Optional cycle stamps of block 0 (compile with -DH2O_PHASE_TIMERS).
#ifdef H2O_PHASE_TIMERS
__device__ long long g_chunk_prof[32];
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

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void key_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kKeyThreads) : "memory"); }

// Byte offset of 16-byte piece `c16` (0..7) of row `row` inside a 128-byte-swizzled block of 128-byte rows.
__device__ __forceinline__ uint32_t swz(int row, int c16) {
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((c16 ^ (row & 7)) << 4));
}

// Eviction candidate; "none" is the largest value of the order, so plain comparisons suffice.
struct Cand {
  unsigned long long key;
  int pos, slot, x;
  float e_next;
};
__device__ __forceinline__ bool cand_before(unsigned long long ka, int pa, unsigned long long kb, int pb) {
  return (ka < kb) | ((ka == kb) & (pa < pb));  // no short-circuit: branch-free
}
__device__ __forceinline__ Cand cand_min(const Cand& a, const Cand& b) { return cand_before(b.key, b.pos, a.key, a.pos) ? b : a; }

template <int N>
__device__ __forceinline__ Cand cand_min_of(const Cand (&c)[N]) {  // balanced tree: short dependency chain
  if constexpr (N == 2) {
    return cand_min(c[0], c[1]);
  } else if constexpr (N == 4) {
    return cand_min(cand_min(c[0], c[1]), cand_min(c[2], c[3]));
  } else {
    static_assert(N == 8, "keys per thread");
    return cand_min(cand_min(cand_min(c[0], c[1]), cand_min(c[2], c[3])),
                    cand_min(cand_min(c[4], c[5]), cand_min(c[6], c[7])));
  }
}

// Wait for the tensor-memory loads in flight; the registers are named so that no use moves above the wait.
template <int N>
__device__ __forceinline__ void tmem_wait_ld_regs(uint32_t (&r)[N]) {
  if constexpr (N == 2) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]), "+r"(r[1])::"memory");
  } else if constexpr (N == 4) {
    tmem_wait_ld4(r[0], r[1], r[2], r[3]);
  } else {
    static_assert(N == 8, "keys per thread");
    tmem_wait_ld8(r[0], r[1], r[2], r[3], r[4], r[5], r[6], r[7]);
  }
}

// KT = keys per thread = most 128-key tiles a unit of this cache can need.
template <int KT>
__global__ void __launch_bounds__(kThreads, KT <= 2 ? 3 : 2)
decode_chunk_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, CacheView c, const __nv_bfloat16* __restrict__ k_in,
                    const __nv_bfloat16* __restrict__ v_in, __nv_bfloat16* __restrict__ out,
                    int32_t* __restrict__ evicted_pos, int tok0, int n_tok, int tiles_cap, int unit_base) {
  extern __shared__ unsigned char dyn_raw[];
  __shared__ Shared sh;
  constexpr int kBatchTiles = batch_tiles(KT);
  constexpr int res_tiles = kBatchTiles;
  unsigned char* dyn = dyn_raw + ((1024u - (smem_u32(dyn_raw) & 1023u)) & 1023u);
  unsigned char* kv = dyn;                                        // one batch of key tiles, later of value tiles
  unsigned char* p_hi = kv + res_tiles * kTileBytes;              // [2 blocks of 64 keys per tile][kC tokens][128 B]
  unsigned char* p_lo = p_hi + res_tiles * 2 * kPBlockBytes;
  unsigned char* q_s = p_lo + res_tiles * 2 * kPBlockBytes;       // [2 halves][kC tokens][128 B]
  const uint32_t col_o = (uint32_t)(tiles_cap * kC);              // O^T: kC columns behind the scores
  const uint32_t ncols = tmem_cols(tiles_cap);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int su = unit_base + (int)blockIdx.x;  // launch position of the unit
  const UnitMeta mt = c.meta[su];
  const int u = mt.unit, r = mt.rwin, B = mt.kbud + mt.rwin;
  const int cnt0 = c.count[su], t0 = c.tpos[su];
  const int ceff = min(kC, n_tok - tok0);
  const int nk = cnt0 + ceff;                          // keys in play: cached entries, then the chunk's own
  const int ntiles = (nk + kTileRows - 1) / kTileRows;
  const int nbatch = (ntiles + kBatchTiles - 1) / kBatchTiles;
  if (ntiles > tiles_cap || tiles_cap > KT || ceff < 1) {                // the host never launches this; leave before any barrier exists
    if (tid == 0) atomicCAS(c.status, 0, H2O_ERR_STATE);
    return;
  }
  const int64_t in_stride = (int64_t)c.units * kD;     // elements between consecutive tokens of the inputs
  const __nv_bfloat16* k_u = k_in + ((int64_t)tok0 * c.units + u) * kD;
  const __nv_bfloat16* v_u = v_in + ((int64_t)tok0 * c.units + u) * kD;

  if (tid == 0) {
    for (int b = 0; b < kMaxBatches; ++b) {
      mbar_init(&sh.k_full[b], 1);
      mbar_init(&sh.k_ready[b], kKeyThreads);
      mbar_init(&sh.s_done[b], 1);
      mbar_init(&sh.v_full[b], 1);
      mbar_init(&sh.p_ready[b], kKeyThreads);
      mbar_init(&sh.o_done[b], 1);
    }
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kKeyWarps) tmem_alloc(&sh.tmem_base, ncols);
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
    }
    // S^T = K Q^T, one batch of key tiles at a time
    for (int b = 0; b < nbatch; ++b) {
      const int tb = min(kBatchTiles, ntiles - b * kBatchTiles);
      if (b > 0) ok = ok && wait_or_abort(&sh.s_done[b - 1], 0, abort_flag);  // the previous batch has been read
      ok = __all_sync(0xffffffffu, ok);
      if (ok && lane == 0) {
        mbar_expect_tx(&sh.k_full[b], (uint32_t)(tb * kTileBytes + (b == 0 ? 2 * kQHalfBytes : 0)));
        if (b == 0) {
          tma_load_3d(q_s, &map_q, 0, u, tok0, &sh.k_full[0]);
          tma_load_3d(q_s + kQHalfBytes, &map_q, 64, u, tok0, &sh.k_full[0]);
        }
        for (int ml = 0; ml < tb; ++ml) {
          const int row = (int)mt.slot_off + (b * kBatchTiles + ml) * kTileRows;
          tma_load_3d(kv + ml * kTileBytes, &map_k, 0, 0, row, &sh.k_full[b]);
          tma_load_3d(kv + ml * kTileBytes + kHalfBytes, &map_k, 64, 0, row, &sh.k_full[b]);
        }
      }
      // ... once the key threads have put the chunk's own keys behind the cached ones
      ok = ok && wait_or_abort(&sh.k_ready[b], 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      if (ok && elect_one()) {
        constexpr uint32_t idesc_s = instr_desc_f16(kTileRows, kC, kFmtBF16, kFmtBF16, false, false);
        const uint32_t a0 = smem_u32(kv), b0 = smem_u32(q_s);
        for (int ml = 0; ml < tb; ++ml) {
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks) {
            const uint32_t offa = (uint32_t)ml * kTileBytes + (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
            const uint32_t offb = (uint32_t)(ks >> 2) * kQHalfBytes + (uint32_t)(ks & 3) * 32u;
            mma_ss(tmem + kColS + (uint32_t)((b * kBatchTiles + ml) * kC), smem_desc_sw128(a0 + offa, 16, 1024),
                   smem_desc_sw128(b0 + offb, 16, 1024), idesc_s, ks > 0);
          }
        }
        mma_commit(&sh.s_done[b]);
      }
      __syncwarp();
    }
    // the key tiles are dead once the scores exist: the values take their place, batch by batch;
    // O^T += V^T P^T (hi and lo halves of P) for each batch once its probabilities are staged
    for (int b = 0; b < nbatch; ++b) {
      const int tb = min(kBatchTiles, ntiles - b * kBatchTiles);
      ok = ok && wait_or_abort(b == 0 ? &sh.s_done[nbatch - 1] : &sh.o_done[b - 1], 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok && lane == 0) {
        mbar_expect_tx(&sh.v_full[b], (uint32_t)(tb * kTileBytes));
        for (int ml = 0; ml < tb; ++ml) {
          const int row = (int)mt.slot_off + (b * kBatchTiles + ml) * kTileRows;
          tma_load_3d(kv + ml * kTileBytes, &map_v, 0, 0, row, &sh.v_full[b]);
          tma_load_3d(kv + ml * kTileBytes + kHalfBytes, &map_v, 64, 0, row, &sh.v_full[b]);
        }
      }
      ok = ok && wait_or_abort(&sh.p_ready[b], 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      if (ok && elect_one()) {
        constexpr uint32_t idesc_o = instr_desc_f16(kD, kC, kFmtBF16, kFmtBF16, true, false);
        const uint32_t v0 = smem_u32(kv), ph = smem_u32(p_hi), pl = smem_u32(p_lo);
        for (int kb = 0; kb < 2 * tb; ++kb) {
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint32_t offv = (uint32_t)(kb >> 1) * kTileBytes + (uint32_t)(((kb & 1) * 64 + ks * 16) * 128);
            const uint32_t offp = (uint32_t)kb * kPBlockBytes + (uint32_t)ks * 32u;
            const uint64_t da = smem_desc_sw128(v0 + offv, kHalfBytes, 1024);
            mma_ss(tmem + col_o, da, smem_desc_sw128(ph + offp, 16, 1024), idesc_o, b > 0 || kb > 0 || ks > 0);
            mma_ss(tmem + col_o, da, smem_desc_sw128(pl + offp, 16, 1024), idesc_o, true);
          }
        }
        mma_commit(&sh.o_done[b]);
      }
      __syncwarp();
    }
  } else {
    // ---------------- key threads: thread (warp, lane) owns keys 128 m + 32 warp + lane ----------------
    const int x0 = tid;  // key of tile 0; also this thread's TMEM lane
    bool ok = true;
    bool alive[KT];
    double acc[KT];
    int pos[KT], slot[KT], jx[KT];
#pragma unroll
    for (int m = 0; m < KT; ++m) {
      const int x = m * kTileRows + x0;
      alive[m] = x < cnt0;
      acc[m] = 0.0;
      pos[m] = 0;
      slot[m] = x;
      jx[m] = x - cnt0;  // index inside the chunk (if 0 <= jx < ceff)
      if (alive[m]) {
        acc[m] = c.acc[mt.slot_off + x];
        pos[m] = c.pos[mt.slot_off + x];
      } else if (jx[m] < ceff) {  // one of the chunk's own keys: enters the set at token jx with an empty score
        pos[m] = t0 + jx[m];
        slot[m] = -1;
      }
    }
    // rows [cnt0, cnt0 + ceff) of the key / value matrices are the chunk's own: written behind the
    // cached rows in the layout the TMA produced; rows no key owns are zeroed (values only)
    auto patch_rows = [&](const __nv_bfloat16* src_u, int b, bool zero_tail) {
      const int row_lo = b * kBatchTiles * kTileRows, row_hi = row_lo + kBatchTiles * kTileRows;
      for (int idx = tid; idx < ceff * 16; idx += kKeyThreads) {
        const int j = idx >> 4, c16 = idx & 15;
        const int row = cnt0 + j;
        if (row >= row_lo && row < row_hi) {
          const uint4 val = *reinterpret_cast<const uint4*>(src_u + (int64_t)j * in_stride + c16 * 8);
          const int rl = row - row_lo;
          unsigned char* dst = kv + (rl >> 7) * kTileBytes + (c16 >> 3) * kHalfBytes + swz(rl & 127, c16 & 7);
          *reinterpret_cast<uint4*>(dst) = val;
        }
      }
      if (zero_tail) {
        const int z_lo = max(nk, row_lo), z_hi = min(ntiles * kTileRows, row_hi);
        for (int idx = tid; idx < (z_hi - z_lo) * 16; idx += kKeyThreads) {
          const int rl = z_lo + (idx >> 4) - row_lo, z16 = idx & 15;
          unsigned char* dst = kv + (rl >> 7) * kTileBytes + (z16 >> 3) * kHalfBytes + swz(rl & 127, z16 & 7);
          *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    };
    DC_STAMP(0);
    for (int b = 0; b < nbatch; ++b) {
      ok = wait_or_abort(&sh.k_full[b], 0, abort_flag) && ok;
      patch_rows(k_u, b, false);
      fence_proxy_async();
      mbar_arrive(&sh.k_ready[b]);
    }
    DC_STAMP(1);

    // ---- scores -> exponentials, in place in tensor memory ----
    // Everything that walks the tokens below is a ROLLED loop over tensor-memory columns: straight-line
    // code that runs once per token would be bound by instruction fetch, not by the arithmetic.
    ok = wait_or_abort(&sh.s_done[nbatch - 1], 0, abort_flag) && ok;
    ok = __all_sync(0xffffffffu, ok);
    DC_STAMP(2);
    tc_fence_after();
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    // Reference maximum of every token's row: over all keys of that row, alive or not — any reference
    // gives the same softmax, and this one needs no reduction inside the sequential loop.  Should a key
    // that died earlier in the chunk tower so far above the live ones that their exponentials vanish,
    // the row falls back to the live maximum (two extra exchanges, see `rescue` below).
    // Scores are kept in the base-2 domain, times c log2(e) rounded once as in the prefill kernels.
    const float scale2 = c.scale * 1.4426950408889634f;
    if (ok) {
      float mx[kC];
#pragma unroll
      for (int i = 0; i < kC; ++i) mx[i] = -INFINITY;
      for (int m = 0; m < ntiles; ++m) {
        uint32_t raw[32];
        tmem_ld32(tmem + kColS + (uint32_t)(m * kC) + lane_base, raw);
        tmem_wait_ld();
        const int jxm = m * kTileRows + x0 - cnt0;
        // a key takes part in token i's row if it is cached or one of the chunk's keys 0..i
        const int first = jxm < 0 ? 0 : (jxm < ceff ? jxm : kC);
#pragma unroll
        for (int i = 0; i < kC; ++i) mx[i] = fmaxf(mx[i], i >= first ? __uint_as_float(raw[i]) : -INFINITY);
      }
      float mine = -INFINITY;
#pragma unroll
      for (int i = 0; i < kC; ++i) {
        const float v = warp_max(mx[i]);
        if (lane == i) mine = v;
      }
      sh.wmax[warp][lane] = mine;
    }
    key_sync();
    if (tid < kC)  // the scale is positive, so the largest scaled score is the scaled largest raw score
      sh.m_row[tid] = scale2 * fmaxf(fmaxf(sh.wmax[0][tid], sh.wmax[1][tid]), fmaxf(sh.wmax[2][tid], sh.wmax[3][tid]));
    key_sync();
    if (ok) {
      for (int m = 0; m < ntiles; ++m) {
        uint32_t raw[32];
        tmem_ld32(tmem + kColS + (uint32_t)(m * kC) + lane_base, raw);
        tmem_wait_ld();
        const int jxm = m * kTileRows + x0 - cnt0;
        const int first = jxm < 0 ? 0 : (jxm < ceff ? jxm : kC);
#pragma unroll
        for (int i = 0; i < kC; ++i)  // scaled score; -inf where the key is not part of the row
          raw[i] = __float_as_uint(i >= first ? __uint_as_float(raw[i]) * scale2 : -INFINITY);
        tmem_st32(tmem + kColS + (uint32_t)(m * kC) + lane_base, raw);
      }
      tmem_wait_st();
    }
    DC_STAMP(3);

    // ---- the tokens, in order (Algorithm 1) ----
    int live = cnt0;  // entries in the cache before the current token
    float l;
    // this thread's keys: exponentials in the current token's row, scaled scores of the next row and of
    // the row after next (in flight)
    float e_cur[KT];
    uint32_t nxt[KT], nn[KT];
    // Live-maximum fallback for row `row` (scores `tv`): exponentials `ev` relative to the largest score
    // among the entries alive in that row, and their sum.  Reached by all key threads together.
    auto rescue = [&](const uint32_t (&tv)[KT], float (&ev)[KT], int row) -> float {
      float mx = -INFINITY;
#pragma unroll
      for (int m = 0; m < KT; ++m)
        if (alive[m] | (jx[m] == row)) mx = fmaxf(mx, __uint_as_float(tv[m]));
      mx = warp_max(mx);
      if (lane == 0) sh.redo[warp] = mx;
      key_sync();
      const float ml = fmaxf(fmaxf(sh.redo[0], sh.redo[1]), fmaxf(sh.redo[2], sh.redo[3]));
      float s2 = 0.f;
#pragma unroll
      for (int m = 0; m < KT; ++m) {
        ev[m] = ex2(__uint_as_float(tv[m]) - ml);
        if (alive[m] | (jx[m] == row)) s2 += ev[m];
      }
      s2 = warp_sum(s2);
      if (lane == 0) sh.redo2[warp] = s2;
      key_sync();
      return (sh.redo2[0] + sh.redo2[1]) + (sh.redo2[2] + sh.redo2[3]);
    };
    constexpr float kTinySum = 1e-30f;  // below this the live exponentials have (nearly) underflowed
    {
      uint32_t t0v[KT];
#pragma unroll
      for (int m = 0; m < KT; ++m) {
        t0v[m] = 0xff800000u;  // -inf
        nxt[m] = 0xff800000u;
        if (ok && m < ntiles) {
          tmem_ld1(tmem + kColS + (uint32_t)(m * kC) + lane_base, t0v[m]);
          if (ceff > 1) tmem_ld1(tmem + kColS + (uint32_t)(m * kC) + 1u + lane_base, nxt[m]);
        }
      }
      tmem_wait_ld_regs(t0v);
      tmem_wait_ld_regs(nxt);
      const float m0 = sh.m_row[0];
#pragma unroll
      for (int m = 0; m < KT; ++m) e_cur[m] = ex2(__uint_as_float(t0v[m]) - m0);
      // normaliser of the first token: nothing has been evicted yet
      float sm = 0.f;
#pragma unroll
      for (int m = 0; m < KT; ++m)
        if (alive[m] | (jx[m] == 0)) sm += e_cur[m];
      sm = warp_sum(sm);
      if (lane == 0) sh.post_sum[1][warp] = sm;
      key_sync();
      const float4 s4 = *reinterpret_cast<const float4*>(sh.post_sum[1]);
      l = (s4.x + s4.y) + (s4.z + s4.w);
      if (!(l > kTinySum)) l = rescue(t0v, e_cur, 0);
    }
#pragma unroll 1
    for (int i = 0; i < ceff; ++i) {
#pragma unroll
      for (int m = 0; m < KT; ++m) {  // the row after next, in flight while this token is worked on
        nn[m] = 0xff800000u;  // -inf: no such row
        if (ok && m < ntiles && i + 2 < ceff) tmem_ld1(tmem + kColS + (uint32_t)(m * kC + i + 2) + lane_base, nn[m]);
      }
      const int t = t0 + i, par = i & 1;
      const float inv_l = __frcp_rn(l);
      const bool full = live >= B;
      Cand cm[KT];
      float en[KT];  // exponentials of the next row
      const float m_next = i + 1 < ceff ? sh.m_row[i + 1] : 0.f;
      float sm = 0.f;
#pragma unroll
      for (int m = 0; m < KT; ++m) {
        en[m] = ex2(__uint_as_float(nxt[m]) - m_next);  // 0 where the key is not part of that row
        alive[m] = alive[m] | (jx[m] == i);  // the token's own key enters the set
        const float p = alive[m] ? e_cur[m] * inv_l : 0.f;
        if (alive[m]) acc[m] += (double)p;  // Algorithm 2: accumulated score
        // the probability replaces the score in tensor memory (zero for dead or unborn keys)
        if (ok && m < ntiles) tmem_st1(tmem + kColS + (uint32_t)(m * kC + i) + lane_base, __float_as_uint(p));
        const bool elig = alive[m] & (pos[m] <= t - r);  // outside the recent window: may be evicted (used when full)
        cm[m].key = elig ? (unsigned long long)__double_as_longlong(acc[m]) : ~0ull;
        cm[m].pos = elig ? pos[m] : INT_MAX;
        cm[m].slot = slot[m];
        cm[m].x = elig ? m * kTileRows + x0 : -1;
        cm[m].e_next = en[m];
        sm += (alive[m] | (jx[m] == i + 1)) ? en[m] : 0.f;  // next row, over the set before this token's eviction
      }
      if (full) {
        // warp minimum under (score, position) and warp sum, interleaved: two independent chains
        const Cand cd = cand_min_of(cm);
        const unsigned hi = (unsigned)(cd.key >> 32), lo = (unsigned)cd.key;
        const unsigned mh = __reduce_min_sync(0xffffffffu, hi);
        sm += __shfl_xor_sync(0xffffffffu, sm, 16);
        const unsigned ml = __reduce_min_sync(0xffffffffu, hi == mh ? lo : 0xffffffffu);
        sm += __shfl_xor_sync(0xffffffffu, sm, 8);
        const bool tie = (cd.x >= 0) & (hi == mh) & (lo == ml);
        const unsigned mp = __reduce_min_sync(0xffffffffu, tie ? (unsigned)cd.pos : 0xffffffffu);
        sm += __shfl_xor_sync(0xffffffffu, sm, 4);
        const unsigned who = __ballot_sync(0xffffffffu, tie & ((unsigned)cd.pos == mp));
        sm += __shfl_xor_sync(0xffffffffu, sm, 2);
        sm += __shfl_xor_sync(0xffffffffu, sm, 1);
        const int src = who ? __ffs(who) - 1 : 0;
        const int w_slot = __shfl_sync(0xffffffffu, cd.slot, src);
        const int w_x = __shfl_sync(0xffffffffu, cd.x, src);
        const float w_en = __shfl_sync(0xffffffffu, cd.e_next, src);
        if (lane == 0) {
          sh.post_key[par][warp] = who ? (((unsigned long long)mh << 32) | ml) : ~0ull;
          sh.post_pos[par][warp] = who ? (int)mp : INT_MAX;
          sh.post_slot[par][warp] = w_slot;
          sh.post_x[par][warp] = who ? w_x : -1;
          sh.post_enext[par][warp] = w_en;
          sh.post_sum[par][warp] = sm;
        }
      } else {
        sm = warp_sum(sm);
        if (lane == 0) sh.post_sum[par][warp] = sm;
      }
      key_sync();
      const float4 s4 = *reinterpret_cast<const float4*>(sh.post_sum[par]);
      const float lsum = (s4.x + s4.y) + (s4.z + s4.w);
      tmem_wait_ld_regs(nn);
      if (full) {
        const ulonglong2 k01 = *reinterpret_cast<const ulonglong2*>(&sh.post_key[par][0]);
        const ulonglong2 k23 = *reinterpret_cast<const ulonglong2*>(&sh.post_key[par][2]);
        const int4 p4 = *reinterpret_cast<const int4*>(sh.post_pos[par]);
        const bool b01 = cand_before(k01.y, p4.y, k01.x, p4.x), b23 = cand_before(k23.y, p4.w, k23.x, p4.z);
        const unsigned long long ka = b01 ? k01.y : k01.x, kb = b23 ? k23.y : k23.x;
        const int pa = b01 ? p4.y : p4.x, pb = b23 ? p4.w : p4.z;
        const int wa = b01 ? 1 : 0, wbi = b23 ? 3 : 2;
        const bool bb = cand_before(kb, pb, ka, pa);
        const int wv = bb ? wbi : wa;
        const int vx = sh.post_x[par][wv];
        float v_en = 0.f;
        if (vx >= 0) {
          const int vslot = sh.post_slot[par][wv];
          v_en = sh.post_enext[par][wv];
#pragma unroll
          for (int m = 0; m < KT; ++m) {
            const bool is_victim = m * kTileRows + x0 == vx;
            alive[m] = alive[m] & !is_victim;
            slot[m] = (!is_victim & (jx[m] == i)) ? vslot : slot[m];  // in-place replacement of the victim
          }
          if (tid == 0) sh.evicted[i] = bb ? pb : pa;
        } else {  // a full cache always has a candidate; record instead of corrupting
#pragma unroll
          for (int m = 0; m < KT; ++m)
            if (jx[m] == i) alive[m] = false;
          if (tid == 0) {
            sh.evicted[i] = -1;
            atomicCAS(c.status, 0, H2O_ERR_STATE);
          }
        }
        l = lsum - v_en;
        if (i + 1 < ceff && v_en > 0.25f * lsum) {  // cancellation would cost digits: sum again without the victim
          float s2 = 0.f;
#pragma unroll
          for (int m = 0; m < KT; ++m)
            if (alive[m] | (jx[m] == i + 1)) s2 += en[m];
          s2 = warp_sum(s2);
          if (lane == 0) sh.redo[warp] = s2;
          key_sync();
          l = (sh.redo[0] + sh.redo[1]) + (sh.redo[2] + sh.redo[3]);
        }
      } else {
#pragma unroll
        for (int m = 0; m < KT; ++m)
          if (jx[m] == i) slot[m] = live;
        live += 1;
        if (tid == 0) sh.evicted[i] = -1;
        l = lsum;
      }
      if (i + 1 < ceff && !(l > kTinySum)) l = rescue(nxt, en, i + 1);
#pragma unroll
      for (int m = 0; m < KT; ++m) {
        e_cur[m] = en[m];
        nxt[m] = nn[m];
      }
    }
    tmem_wait_st();
    DC_STAMP(4);

    // ---- per batch of tiles: probabilities to shared memory as bf16 hi + lo, values patched ----
    for (int b = 0; b < nbatch; ++b) {
      const int tb = min(kBatchTiles, ntiles - b * kBatchTiles);
      if (b > 0) ok = wait_or_abort(&sh.o_done[b - 1], 0, abort_flag) && ok;  // staging and value tiles are free again
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      for (int ml = 0; ml < tb; ++ml) {
        uint32_t pr[32];
        if (ok) {
          tmem_ld32(tmem + kColS + (uint32_t)((b * kBatchTiles + ml) * kC) + lane_base, pr);
          tmem_wait_ld();
        }
        const uint32_t pcol = (uint32_t)((ml * 2 + (x0 >> 6)) * kPBlockBytes + (x0 & 7) * 2);
        const int pc16 = (x0 & 63) >> 3;
#pragma unroll
        for (int i = 0; i < kC; ++i) {
          const float p = (ok && i < ceff) ? __uint_as_float(pr[i]) : 0.f;
          const __nv_bfloat16 hi = __float2bfloat16_rn(p);
          const __nv_bfloat16 lo = __float2bfloat16_rn(p - __bfloat162float(hi));
          const uint32_t off = pcol + (uint32_t)((i >> 3) * 1024 + (i & 7) * 128 + ((pc16 ^ (i & 7)) << 4));
          *reinterpret_cast<__nv_bfloat16*>(p_hi + off) = hi;
          *reinterpret_cast<__nv_bfloat16*>(p_lo + off) = lo;
        }
      }
      ok = wait_or_abort(&sh.v_full[b], 0, abort_flag) && ok;
      patch_rows(v_u, b, true);
      fence_proxy_async();
      mbar_arrive(&sh.p_ready[b]);
    }
    DC_STAMP(6);

    // ---- write the state back: scores of the survivors, the chunk's surviving rows into their slots ----
#pragma unroll
    for (int m = 0; m < KT; ++m) {
      if (alive[m] && H2O_IN_RANGE(slot[m], mt.kbud + mt.rwin, c.status) &&
          H2O_IN_RANGE(mt.slot_off + slot[m], c.total_slots, c.status)) {
        c.acc[mt.slot_off + slot[m]] = acc[m];
        if (jx[m] >= 0) c.pos[mt.slot_off + slot[m]] = pos[m];
      }
      if (jx[m] >= 0 && jx[m] < ceff) sh.wb_slot[jx[m]] = alive[m] ? slot[m] : -1;
    }
    key_sync();
    for (int idx = tid; idx < ceff * 32; idx += kKeyThreads) {
      const int j = idx >> 5, pc = idx & 31, c16 = pc & 15;
      const int sl = sh.wb_slot[j];
      if (sl >= 0 && H2O_IN_RANGE(sl, mt.kbud + mt.rwin, c.status) && H2O_IN_RANGE(mt.slot_off + sl, c.total_slots, c.status)) {
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
    ok = wait_or_abort(&sh.o_done[nbatch - 1], 0, abort_flag) && ok;
    ok = __all_sync(0xffffffffu, ok);
    DC_STAMP(8);
    tc_fence_after();
    if (ok) {
      uint32_t o[32];
      tmem_ld32(tmem + col_o + lane_base, o);
      tmem_wait_ld();
      __nv_bfloat16* out_u = out + ((int64_t)tok0 * c.units + u) * kD + tid;
#pragma unroll
      for (int i = 0; i < kC; ++i)
        if (i < ceff) out_u[(int64_t)i * in_stride] = __float2bfloat16_rn(__uint_as_float(o[i]));
    }
  }
  DC_STAMP(9);
  tc_fence_before();
  __syncthreads();
  DC_STAMP(10);
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
  if (warp == kKeyWarps) {
    tc_fence_after();
    tmem_dealloc(tmem, ncols);
  }
}

}  // namespace

#ifdef H2O_PHASE_TIMERS
extern "C" int h2o_debug_chunk_prof(long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_chunk_prof, sizeof(long long) * 32);
}
#endif

bool decode_chunk_supported(int dtype, int head_dim, int max_B, int64_t total_slots) {
  return prefill_tc_supported(dtype, head_dim) && max_B + kC <= kMaxKeys && total_slots < INT_MAX - kTileRows;
}

namespace {

template <int KT>
cudaError_t launch_kt(const CUtensorMap& map_q, const CUtensorMap& map_k, const CUtensorMap& map_v, const CacheView& c,
                      const void* k, const void* v, int tok0, int n_tokens, void* out, int32_t* evicted_pos,
                      int tiles_cap, int unit_base, int n_units, cudaStream_t stream) {
  static unsigned long long attr_flags = 0;  // one word per template instance, one bit per device
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_chunk_kernel<KT>), dyn_smem_bytes(KT),
                                        &attr_flags);
    if (e != cudaSuccess) return e;
  }
  decode_chunk_kernel<KT><<<(unsigned)n_units, kThreads, dyn_smem_bytes(KT), stream>>>(
      map_q, map_k, map_v, c, static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v),
      static_cast<__nv_bfloat16*>(out), evicted_pos, tok0, n_tokens, tiles_cap, unit_base);
  return cudaGetLastError();
}

int tiles_for(int B) { return (B + kC + kTileRows - 1) / kTileRows; }

}  // namespace

// `meta` is the host copy of the unit table, in launch order (largest budget first).  Units are
// grouped by the keys per thread their budget needs, one grid per group and chunk: a unit with a
// small budget then neither pays for eight keys per thread nor for one block per SM.
cudaError_t launch_decode_chunk(const CacheView& c, int64_t total_slots, const UnitMeta* meta, const void* q,
                                const void* k, const void* v, int n_tokens, void* out, int32_t* evicted_pos,
                                cudaStream_t stream) {
  CUtensorMap map_q, map_k, map_v;
  if (!make_tile_map(&map_q, q, n_tokens, c.units, kC) || !make_tile_map(&map_k, c.K, total_slots, 1, kTileRows) ||
      !make_tile_map(&map_v, c.V, total_slots, 1, kTileRows))
    return cudaErrorInvalidValue;
  int n8 = 0, n4 = 0;  // units needing more than 4 tiles, then more than 2
  for (int su = 0; su < c.units; ++su) {
    const int t = tiles_for(meta[su].kbud + meta[su].rwin);
    if (t > kMaxTiles) return cudaErrorInvalidValue;
    n8 += t > 4;
    n4 += t > 2 && t <= 4;
  }
  const int n2 = c.units - n8 - n4;
  for (int tok0 = 0; tok0 < n_tokens; tok0 += kC) {
    cudaError_t e = cudaSuccess;
    if (n8 > 0)
      e = launch_kt<8>(map_q, map_k, map_v, c, k, v, tok0, n_tokens, out, evicted_pos,
                       tiles_for(meta[0].kbud + meta[0].rwin), 0, n8, stream);
    if (e == cudaSuccess && n4 > 0)
      e = launch_kt<4>(map_q, map_k, map_v, c, k, v, tok0, n_tokens, out, evicted_pos,
                       tiles_for(meta[n8].kbud + meta[n8].rwin), n8, n4, stream);
    if (e == cudaSuccess && n2 > 0)
      e = launch_kt<2>(map_q, map_k, map_v, c, k, v, tok0, n_tokens, out, evicted_pos,
                       tiles_for(meta[n8 + n4].kbud + meta[n8 + n4].rwin), n8 + n4, n2, stream);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace h2o
