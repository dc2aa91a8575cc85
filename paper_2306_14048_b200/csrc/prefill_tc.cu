// Prompt attention on the tensor cores (bf16, head_dim 128): tcgen05.mma with TMEM
// accumulators, operands staged in shared memory by TMA, warp-specialised roles.
//
// Column sums (this file, first kernel).  acc0[j] = sum_{i >= j} exp(c q_i.k_j - lse_i) needs the
// final row normalisers, so scores are recomputed after the forward pass.  The kernel is
// K-stationary and computes the TRANSPOSED tile S^T = K_j Q_i^T: a TMEM lane (= one thread of the
// epilogue) then owns one key column j and sums over queries in registers — no atomics, fixed
// order, reproducible.  A thread block takes key block j and its mirror nb-1-j, so every block
// does the same number of tiles of the causal triangle.
//
// Paper: accumulated attention score of Algorithm 2 evaluated over all prompt rows (the prefill
// branch of the Appendix A pseudocode).
#include <algorithm>
#include <cstring>

#include "h2o_internal.cuh"
#include "sm100_ptx.cuh"

namespace h2o {

namespace {

using namespace ptx;

constexpr int kD = 128;           // head_dim handled here
constexpr int kTile = 128;        // rows of a Q / K tile
constexpr int kBoxBytes = kTile * 128;   // one TMA box: 128 rows x 64 bf16
constexpr int kTileBytes = 2 * kBoxBytes;  // two boxes cover head_dim 128
constexpr double kLog2eD = 1.4426950408889634074;

// Optional cycle accounting of the forward kernel's softmax loop (compile with -DH2O_PHASE_TIMERS).
#ifdef H2O_PHASE_TIMERS
__device__ unsigned long long g_fwd_prof[8];
__device__ long long g_fwd_tl[2][40][10];  // block (0, units-1): per group and tile, clock64 at ten events
#define FWD_TL(g, j, e) do { if (tl_on_ && (j) < 40) g_fwd_tl[g][j][e] = clock64(); } while (0)
#define FWD_CLK(v) const long long v = clock64()
#define FWD_ADD(i, a, b) prof_[i] += (b) - (a)
#else
#define FWD_CLK(v) do { } while (0)
#define FWD_ADD(i, a, b) do { } while (0)
#define FWD_TL(g, j, e) do { } while (0)
#endif

// 32 output columns of one query row: accumulator values times 1 / row sum, as bf16.  A thread owns a row, so
// a warp's store instruction touches 32 different rows; 32-byte stores (whole sectors) halve the number of
// instructions and transactions against 16-byte ones.  `wide` = the output base is 32-byte aligned.
__device__ __forceinline__ void store_out_32(__nv_bfloat16* dst, const uint32_t (&o)[32], float inv_l, bool wide) {
  if (wide) {
#pragma unroll
    for (int c16 = 0; c16 < 2; ++c16) {
      uint32_t w[8];
#pragma unroll
      for (int e = 0; e < 8; ++e)
        w[e] = Vec16<__nv_bfloat16>::pack2(__uint_as_float(o[c16 * 16 + 2 * e]) * inv_l,
                                           __uint_as_float(o[c16 * 16 + 2 * e + 1]) * inv_l);
      st_global_256(dst + c16 * 16, w);
    }
  } else {
#pragma unroll
    for (int c8 = 0; c8 < 4; ++c8) {
      float f[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(o[c8 * 8 + e]) * inv_l;
      Vec16<__nv_bfloat16>::store(dst + c8 * 8, f);
    }
  }
}

// ---- abortable waits: the first role that times out raises a flag every other wait observes ----
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// exp2 of two values on the FMA pipe (packed fp32x2 instructions of this architecture), for a fixed
// share of the column-sum exponentials: the special-function unit delivers only 16 results per clock
// and SM.  Round to nearest integer with the 1.5 * 2^23 trick, degree-5 minimax polynomial of 2^f on
// [-0.5, 0.5] (relative error 1.8e-7 in fp32, the same class as ex2.approx), exponent added with
// integer arithmetic.  Arguments below -126 (rows past the end have -inf) give ~1e-38 instead of 0.
__device__ __forceinline__ float2 ex2_fma2(float2 x) {
  x.x = fmaxf(x.x, -126.f);
  x.y = fmaxf(x.y, -126.f);
  const float2 t = __fadd2_rn(x, make_float2(12582912.f, 12582912.f));
  const float2 n = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
  float2 p = make_float2(0.0013280353741720319f, 0.0013280353741720319f);
  p = __ffma2_rn(p, f, make_float2(0.009675574488937855f, 0.009675574488937855f));
  p = __ffma2_rn(p, f, make_float2(0.05550701171159744f, 0.05550701171159744f));
  p = __ffma2_rn(p, f, make_float2(0.24022118747234344f, 0.24022118747234344f));
  p = __ffma2_rn(p, f, make_float2(0.6931470036506653f, 0.6931470036506653f));
  p = __ffma2_rn(p, f, make_float2(1.0000001192092896f, 1.0000001192092896f));
  return make_float2(__uint_as_float(__float_as_uint(p.x) + (__float_as_uint(t.x) << 23)),
                     __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(t.y) << 23)));
}

// ---------------------------------------------------------------------------------------------
// Column sums
// ---------------------------------------------------------------------------------------------
constexpr int kCsThreads = 320;  // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..9: epilogue
constexpr int kCsQStages = 2;
constexpr int kCsTmemCols = 256;  // two accumulator buffers of 128 columns
constexpr int kCsStatBufs = 8;    // buffers of per-query statistics (at least five, see CsShared)
constexpr int kCsPersistentTiles = 8;  // items of at most this many tiles are walked by persistent blocks

struct CsShared {
  uint64_t k_full, k_empty;
  uint64_t q_full[kCsQStages], q_empty[kCsQStages];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t nl_full[kCsStatBufs];  // the producer warp has staged a tile's row statistics
  uint64_t ps_full, ps_empty;  // hand-over of the second query half's partial sums
  uint32_t tmem_base;
  int abort_flag;
  // per query of the tile: -(reference maximum + log2 of the row sum), log2 domain
  // Filled by the producer warp ahead of the epilogue.  No barrier guards the reuse of a buffer: the producer
  // writes tile t's statistics after Q(t) could be loaded, i.e. after the MMA of tile t-2 completed, which
  // was issued after every epilogue warp had loaded the scores of tile t-4, i.e. finished summing tile t-5.
  __align__(16) float rstat[kCsStatBufs][kTile];
  double psum[kTile];
};

// Work item: one (unit, pair of key blocks {pi, nb-1-pi}); all items of a unit have nb+1 tiles.  A block
// walks over items blockIdx.x, blockIdx.x + gridDim.x, ...: barriers, tensor memory and the pipeline stay
// up from one item to the next, so an item's first loads overlap the previous item's last tiles.
// Grouped-query attention (group > 1): a key block of K/V head h meets the query blocks of all the group's query
// heads h * group + g, one after the other, and their probabilities add up in the same column sums; the tiles of
// a key block are then numbered g * (query blocks) + (query block).
struct CsItem {
  int h, lo, n;   // K/V head, first token and length of the sequence
  int jb0, jb1;   // the two key blocks (jb1 == jb0: one)
  int t0, total;  // tiles of the first key block, tiles of the item
  int nb, group;  // query blocks of the sequence, query heads per K/V head
};
struct CsWalk {
  int w, t;  // item, tile inside the item
  CsItem it;
  __device__ __forceinline__ int jb() const { return t < it.t0 ? it.jb0 : it.jb1; }                       // key block
  __device__ __forceinline__ int local() const { return t < it.t0 ? t : t - it.t0; }  // tile inside its key block
  __device__ __forceinline__ int g() const { return it.group == 1 ? 0 : local() / (it.nb - jb()); }     // query head of the group
  __device__ __forceinline__ int ib() const {                                                             // query block
    return it.group == 1 ? jb() + local() : jb() + local() % (it.nb - jb());
  }
  __device__ __forceinline__ int qh() const { return it.h * it.group + g(); }                             // query head
  __device__ __forceinline__ bool first_of_cb() const { return t == 0 || t == it.t0; }
  __device__ __forceinline__ bool last_of_cb() const { return t == it.t0 - 1 || t == it.total - 1; }
};
__device__ __forceinline__ bool cs_item(const PrefillScratch& s, int n_heads, int max_pairs, int w, CsItem& it) {
  const int u = w / max_pairs, pi = w % max_pairs;
  const int seq = u / n_heads;
  it.h = u % n_heads;
  it.lo = s.cu[seq];
  it.n = s.cu[seq + 1] - it.lo;
  const int nb = (it.n + kTile - 1) / kTile;
  if (pi >= (nb + 1) / 2) return false;
  it.jb0 = pi;
  it.jb1 = nb - 1 - pi;
  it.nb = nb;
  it.t0 = it.group * (nb - it.jb0);  // tiles of key block jb: query blocks jb .. nb-1 of every query head
  it.total = it.t0 + (it.jb1 > it.jb0 ? it.group * (nb - it.jb1) : 0);
  return true;
}
__device__ __forceinline__ bool cs_seek(const PrefillScratch& s, int n_heads, int max_pairs, int n_items, CsWalk& k) {
  while (k.w < n_items && !cs_item(s, n_heads, max_pairs, k.w, k.it)) k.w += (int)gridDim.x;
  return k.w < n_items;
}
__device__ __forceinline__ bool cs_first(const PrefillScratch& s, int n_heads, int max_pairs, int n_items, int group,
                                         CsWalk& k) {
  k.w = (int)blockIdx.x;
  k.t = 0;
  k.it.group = group;
  return cs_seek(s, n_heads, max_pairs, n_items, k);
}
__device__ __forceinline__ bool cs_next(const PrefillScratch& s, int n_heads, int max_pairs, int n_items, CsWalk& k) {
  if (++k.t < k.it.total) return true;
  k.t = 0;
  k.w += (int)gridDim.x;
  return cs_seek(s, n_heads, max_pairs, n_items, k);
}

__global__ void __launch_bounds__(kCsThreads, 2)
colsum_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 PrefillScratch s, int n_heads, int group, int max_pairs, int n_items, float scale2, int32_t* status) {
  extern __shared__ unsigned char dyn_raw[];
  __shared__ CsShared sh;
  unsigned char* dyn = dyn_raw + ((1024u - (smem_u32(dyn_raw) & 1023u)) & 1023u);
  unsigned char* k_tile = dyn;                       // [2 boxes][128 rows][128 B]
  unsigned char* q_ring = dyn + kTileBytes;          // [stages][2 boxes][128 rows][128 B]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(&sh.k_full, 1);
    mbar_init(&sh.k_empty, 1);
    for (int i = 0; i < kCsQStages; ++i) {
      mbar_init(&sh.q_full[i], 1);
      mbar_init(&sh.q_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh.acc_full[i], 1);
      mbar_init(&sh.acc_empty[i], 8);  // one arrival per epilogue warp
    }
    for (int i = 0; i < kCsStatBufs; ++i) mbar_init(&sh.nl_full[i], 1);
    mbar_init(&sh.ps_full, 128);
    mbar_init(&sh.ps_empty, 128);
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, kCsTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;
  // every role walks over the same tiles; g counts them (ring stages, buffers and barrier phases follow g)

  if (warp == 0) {
    // ---------------- producer: row statistics of each query tile (whole warp), TMA loads (lane 0) ----------------
    // P[i][j] = 2^(c2 s - m_i) / l_i = 2^(c2 s - (m_i + log2 l_i)): the normaliser is folded into the
    // exponent's offset, one float per query and no multiplication per score
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
    }
    auto fetch = [&](const CsWalk& k, float2 (&raw)[4]) {  // {m, 1 / l} of the tile's 128 queries, four per lane
      const float2* rowstat = s.rowstat + (int64_t)k.qh() * s.total_tokens + k.it.lo;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int qi = k.ib() * kTile + i * 32 + lane;
        raw[i] = qi < k.it.n ? rowstat[qi] : make_float2(INFINITY, 1.f);  // rows past the end: exp2(-inf) = 0
      }
    };
    CsWalk cur;
    bool have = cs_first(s, n_heads, max_pairs, n_items, group, cur);
    float2 raw[4];
    if (have) fetch(cur, raw);
    bool ok = true;
    for (int g = 0, kc = 0; have && ok; ++g) {
      const bool new_k = cur.first_of_cb();
      if (lane == 0) {
        if (new_k) {
          // the single K buffer: the previous key block's last MMA must have read it
          if (kc >= 1) ok = wait_or_abort(&sh.k_empty, (uint32_t)(kc - 1) & 1u, abort_flag);
          if (ok) {
            mbar_expect_tx(&sh.k_full, kTileBytes);
            tma_load_tile(k_tile, &map_k, cur.it.h, cur.it.lo + cur.jb() * kTile, &sh.k_full);
          }
        }
        const int st = g % kCsQStages;
        ok = ok && wait_or_abort(&sh.q_empty[st], ((uint32_t)(g / kCsQStages) & 1u) ^ 1u, abort_flag);
        if (ok) {
          unsigned char* dst = q_ring + st * kTileBytes;
          mbar_expect_tx(&sh.q_full[st], kTileBytes);
          tma_load_tile(dst, &map_q, cur.qh(), cur.it.lo + cur.ib() * kTile, &sh.q_full[st]);
        }
      }
      if (new_k) ++kc;
      // row statistics of this tile (fetched one iteration ago)
      const int b8 = g % kCsStatBufs;
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
#pragma unroll
      for (int i = 0; i < 4; ++i) sh.rstat[b8][i * 32 + lane] = log2f(raw[i].y) - raw[i].x;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.nl_full[b8]);
      have = cs_next(s, n_heads, max_pairs, n_items, cur);
      if (have) fetch(cur, raw);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (whole warp runs the loop, one elected lane issues) ----------------
    constexpr uint32_t idesc = instr_desc_f16(kTile, kTile, kFmtBF16, kFmtBF16, false, false);
    CsWalk cur;
    bool have = cs_first(s, n_heads, max_pairs, n_items, group, cur);
    for (int g = 0, kc = 0; have; ++g) {
      bool ok = true;
      if (cur.first_of_cb()) {
        ok = wait_or_abort(&sh.k_full, (uint32_t)kc & 1u, abort_flag);
        ++kc;
      }
      const int st = g % kCsQStages, b = g & 1;
      // the tile's row statistics must be staged before its scores are handed to the epilogue: the
      // epilogue waits for acc_full only (each wait stalls its warps ~200 cycles behind the exponentials)
      ok = ok && wait_or_abort(&sh.nl_full[g % kCsStatBufs], (uint32_t)(g / kCsStatBufs) & 1u, abort_flag);
      ok = ok && wait_or_abort(&sh.q_full[st], (uint32_t)(g / kCsQStages) & 1u, abort_flag);
      ok = ok && wait_or_abort(&sh.acc_empty[b], ((uint32_t)(g >> 1) & 1u) ^ 1u, abort_flag);
      if (!__all_sync(0xffffffffu, ok)) break;
      tc_fence_after();
      const uint32_t a0 = smem_u32(k_tile), b0 = smem_u32(q_ring + st * kTileBytes);
      if (elect_one()) {
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t off = (uint32_t)(ks >> 2) * kBoxBytes + (uint32_t)(ks & 3) * 32u;
          mma_ss(tmem + (uint32_t)b * kTile, smem_desc_sw128(a0 + off, 16, 1024), smem_desc_sw128(b0 + off, 16, 1024),
                 idesc, ks > 0);
        }
        mma_commit(&sh.q_empty[st]);   // the Q stage may be refilled once these MMAs have read it
        mma_commit(&sh.acc_full[b]);   // and the accumulator is ready for the epilogue
        if (cur.last_of_cb()) mma_commit(&sh.k_empty);
      }
      __syncwarp();
      have = cs_next(s, n_heads, max_pairs, n_items, cur);
    }
  } else {
    // ---------------- epilogue: exp and in-thread column sums ----------------
    // Eight warps: warps w and w+4 share a TMEM lane quarter (the same 32 key rows); the first
    // takes queries 0..63 of the tile, the second queries 64..127.
    const int e = threadIdx.x - 64;          // 0..255
    const int quarter = warp & 3;            // TMEM lane quarter this warp may access
    const int half = e >> 7;                 // which 64 queries of the tile
    const int row = quarter * 32 + lane;     // key row inside the tile = TMEM lane
    double total_sum = 0.0;
    bool ok = true;
    CsWalk cur;
    bool have = cs_first(s, n_heads, max_pairs, n_items, group, cur);
    for (int g = 0, cbc = 0; have && ok; ++g) {  // cbc: key blocks finished so far
      const int b = g & 1;
      const int b8 = g % kCsStatBufs;                // buffer of the row statistics
      // One wait per tile: it costs ~200 cycles even when the phase is complete (barrier operations queue
      // behind the exponentials), and testing the barrier early, in the middle of the arithmetic, only moves
      // that stall (the warp issues in order and stops at the first use of the answer).  The row statistics
      // are covered by this wait: the MMA warp saw them staged before it issued the tile.
      ok = wait_or_abort(&sh.acc_full[b], (uint32_t)(g >> 1) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);  // the TMEM loads below are warp-collective
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem + (uint32_t)b * kTile + (uint32_t)half * 64u + ((uint32_t)(quarter * 32) << 16);
      const float4* st4 = reinterpret_cast<const float4*>(&sh.rstat[b8][half * 64]);  // four queries per entry
      uint32_t r0[32], r1[32];
      tmem_ld32(taddr, r0);
      tmem_ld32(taddr + 32u, r1);
      tmem_wait_ld();
      // the scores are in registers: hand the accumulator back before the arithmetic, so that the tile
      // after next is computed (issue latency, 512 tensor cycles, commit) while this one is summed
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.acc_empty[b]);
      float2 sum2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      auto chunk = [&](const uint32_t (&r)[32], int c0, bool masked) {
#pragma unroll
        for (int c4 = 0; c4 < 32; c4 += 4) {
          const float4 st = st4[(c0 + c4) >> 2];
          const float2 xa = __ffma2_rn(make_float2(__uint_as_float(r[c4]), __uint_as_float(r[c4 + 1])),
                                       make_float2(scale2, scale2), make_float2(st.x, st.y));
          const float2 xb = __ffma2_rn(make_float2(__uint_as_float(r[c4 + 2]), __uint_as_float(r[c4 + 3])),
                                       make_float2(scale2, scale2), make_float2(st.z, st.w));
          float2 pa = make_float2(ex2(xa.x), ex2(xa.y));
          float2 pb = ((c4 >> 2) & 1) == 0 ? ex2_fma2(xb) : make_float2(ex2(xb.x), ex2(xb.y));  // a quarter on the FMA pipe
          if (masked) {  // causal: query >= key (diagonal tile only)
            const int ql = half * 64 + c0 + c4;
            if (ql < row) pa.x = 0.f;
            if (ql + 1 < row) pa.y = 0.f;
            if (ql + 2 < row) pb.x = 0.f;
            if (ql + 3 < row) pb.y = 0.f;
          }
          sum2[(c4 >> 2) & 3] = __fadd2_rn(sum2[(c4 >> 2) & 3], __fadd2_rn(pa, pb));
        }
      };
      if (cur.ib() == cur.jb()) {
        chunk(r0, 0, true);
        chunk(r1, 32, true);
      } else {
        chunk(r0, 0, false);
        chunk(r1, 32, false);
      }
      total_sum += (double)(((sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y)) +
                            ((sum2[2].x + sum2[2].y) + (sum2[3].x + sum2[3].y)));
      if (cur.last_of_cb()) {  // last tile of this key block: add the two query halves
        if (half == 1) {
          // the previous key block's partial sums must have been taken
          if (cbc >= 1) ok = wait_or_abort(&sh.ps_empty, (uint32_t)(cbc - 1) & 1u, abort_flag);
          if (ok) {
            sh.psum[row] = total_sum;
            mbar_arrive(&sh.ps_full);
          }
        } else {
          ok = wait_or_abort(&sh.ps_full, (uint32_t)cbc & 1u, abort_flag);
          const int key = cur.jb() * kTile + row;
          if (ok && key < cur.it.n) s.acc0[(int64_t)cur.it.h * s.total_tokens + cur.it.lo + key] = total_sum + sh.psum[row];
          if (ok) mbar_arrive(&sh.ps_empty);
        }
        ok = __all_sync(0xffffffffu, ok);  // keep the warp together for the next tile's collectives
        total_sum = 0.0;
        ++cbc;
      }
      have = cs_next(s, n_heads, max_pairs, n_items, cur);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(status, 0, H2O_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kCsTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Forward: out = softmax(c Q K^T) V over the causal triangle, plus per-row {max, 1/sum}
// ---------------------------------------------------------------------------------------------
// One thread block per (unit, PAIR of 128-query blocks) (short prompts take the persistent kernel further
// down); key tiles of 64, loaded once (TMA) for both query blocks.  One softmax group of four warps per query block (A, B)
// and, per group, two MMA-issuing warps (even key tiles, odd key tiles).  Per group g and key tile j:
//   S_g(j) = Q_g K_j^T           M 128, N 64, K 128; Q and K from shared memory, fp32 accumulator
//                                in TMEM.  Issued two tiles ahead of the softmax, right behind P V(j-2)
//                                by the same thread (the score buffer is the one that product reads).
//   P_g(j) = exp2(c S_g(j) - m)  written by the softmax threads into TMEM as bf16 hi | bf16 lo
//                                (a single bf16 P would put its 2^-9 rounding into the output)
//   O_g   += P_hi V_j + P_lo V_j M 128, N 128, K 64 twice; P is the TMEM operand, V the MN-major
//                                shared-memory operand (with P in shared memory as well the
//                                instruction is bound by shared-memory bandwidth)
// The softmax keeps one thread per query row (row max / sum need no shuffles) and updates the
// reference maximum lazily: O rows in TMEM are rescaled only when the maximum grows by more than
// 8 in the log2 domain.  With two groups, one block per SM: all 512 TMEM columns, 161 KB of shared memory.
// In steady state the tensor pipe is busy about four fifths of the time (S 256 + P V 512 cycles per group
// and tile against a period of ~990), so issue waits behind the other warps' instructions.
// Warps come in groups of four that set their register budget together (setmaxnreg): warps 0..3 TMA and
// MMA issuers (few registers), warps 4..7 softmax of group A (, warps 8..11 softmax of group B, warp 12 the
// fourth MMA issuer, 13..15 idle).  The block starts with 128 registers per thread; the issuers give
// registers back and the softmax warps take them.
__host__ __device__ constexpr int fw_threads(int groups) { return groups == 2 ? 512 : 256; }
constexpr int kFwRegsIssue = 80, kFwRegsSoftmax = 168;
constexpr int kFwKeys = 64;                       // keys per tile
constexpr int kFwKvSlotBytes = 2 * kFwKeys * 128;   // [2 boxes][64 rows][128 B] = 16 KB
constexpr int kFwMaxKvSlots = 6;
// The low halves matter only where a probability is large: a tile whose probabilities all stay below
// kFwLoThreshold of their row's running sum (an upper bound of the final probability) contributes at most
// 2^-9 of them to the output, far inside its tolerance, and its second product is skipped.  The softmax warps
// vote per tile; the decision depends on the data alone, so results stay the same from run to run.
constexpr float kFwLoThreshold = 1.0f / 32.0f;
constexpr bool kFwSplitP = true;                 // P as bf16 hi + bf16 lo (two P V products): one bf16 alone (2^-9 per
                                                 // probability) misses the output tolerance on peaky rows
// Up to this prompt length the persistent one-query-block kernel runs the forward pass (measured: 512-token
// prompts 621 -> 480 us, 2048-token prompts 399 -> 378 us, ragged up to 4096: 13.1 -> 12.4 ms per layer of
// prefill-select); beyond, every block streaming its own K and V through L2 costs more than the fixed costs
// it saves (32768 tokens: 17.2 against 16.0 ms), and two query blocks per thread block share every tile.
constexpr int kFwShortPrompt = 4096;
// ring slots: K_j, V_j, K_j+1, V_j+1 (, K_j+2, V_j+2 with two groups); TMEM columns: O and two S/P buffers per group
__host__ __device__ constexpr int fw_kv_slots(int groups) { return groups == 2 ? 6 : 4; }
__host__ __device__ constexpr uint32_t fw_tmem_cols(int groups) { return groups == 2 ? 512u : 256u; }
constexpr uint32_t kFwColO = 0;                   // O_g : 128 columns each
// S and P share two 64-column buffers per group: S_g(j) lands in buffer j % 2, the softmax reads it into
// registers and writes P_g(j) (bf16 hi in columns 0..31, lo in 32..63) over it, S_g(j+1) meanwhile uses
// the other buffer.  P is thereby double-buffered: the exponentials of tile j+1 need not wait for P V of tile j.
// group g, buffer b: columns 128 G + 128 g + 64 b behind the G output accumulators
constexpr float kRescaleThreshold = 8.0f;

struct FwShared {
  uint64_t q_full[2];
  uint64_t kv_full[kFwMaxKvSlots], kv_empty[kFwMaxKvSlots];
  uint64_t s_full[2][2];  // [group][buffer] MMA -> softmax: S_g(j) complete (one barrier per buffer: two S tiles can be ahead)
  uint64_t p_full[2][2];  // [group][buffer] softmax -> MMA: P_g(j) is in tensor memory
  uint64_t pv_done[2][2]; // [group][tile parity] MMA -> softmax: O_g includes tile j (O_g may be rescaled)
  uint64_t o_final[2];    // MMA -> softmax: O_g includes the group's last tile (a barrier of its own: the softmax
                          // does not wait on every phase of pv_done, so a parity wait for the last one could alias)
  uint32_t tmem_base;
  int abort_flag;
  uint32_t lo_need[2][2][4];  // [group][buffer][softmax warp]: some probability of the tile is large (kFwLoThreshold);
                              // written before the warp's arrival on p_full, read by the issuing warp after its wait
};

// G = query blocks (softmax groups) per thread block.  Two share every K/V tile and fill an SM (all of
// its tensor memory): the instance that is launched.  (One per block works too, two blocks per SM; for
// short prompts the persistent kernel below replaced it.)
template <int G>
__global__ void __launch_bounds__(fw_threads(G), G == 2 ? 1 : 2)
fwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
              const __grid_constant__ CUtensorMap map_v, PrefillScratch s, int n_heads, int kv_div, float scale2,
              __nv_bfloat16* __restrict__ out, int32_t* status) {
  // n_heads counts QUERY heads; query head h reads K/V head h / kv_div (grouped-query attention; 1 otherwise)
  const bool wide_out = (reinterpret_cast<uintptr_t>(out) & 31u) == 0;
  extern __shared__ unsigned char dyn_raw[];
  __shared__ FwShared sh;
  unsigned char* dyn = dyn_raw + ((1024u - (smem_u32(dyn_raw) & 1023u)) & 1023u);
  constexpr int kFwKvSlots = fw_kv_slots(G);
  constexpr uint32_t kFwTmemCols = fw_tmem_cols(G);
  constexpr uint32_t kFwColSP = 128u * G;
  unsigned char* q_tiles = dyn;                       // G x 32 KB
  unsigned char* kv_ring = dyn + G * kTileBytes;      // slots of 16 KB

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#ifdef H2O_PHASE_TIMERS
  const bool tl_on_ = blockIdx.x == 0 && blockIdx.y == 0 && (threadIdx.x & 31) == 0 && ((threadIdx.x >> 5) >= 1 && ((threadIdx.x >> 5) <= 4 || (threadIdx.x >> 5) == 8 || (threadIdx.x >> 5) == 12));
#endif
  const int u = blockIdx.y;
  const int seq = u / n_heads, h = u % n_heads;
  const int lo = s.cu[seq], n = s.cu[seq + 1] - lo;
  const int nb = (n + kTile - 1) / kTile;
  const int nitem = G == 2 ? (nb + 1) / 2 : nb;  // pairs of query blocks, or single ones
  if ((int)blockIdx.x >= nitem) return;
  const int pr = nitem - 1 - (int)blockIdx.x;  // long ones first
  const int ibA = G == 2 ? 2 * pr : pr, ibB = ibA + 1;
  const bool hasB = G == 2 && ibB < nb;
  // key tiles visible to each group (keys 0 .. min(n, (ib+1)*128) - 1)
  const int ntA = (min(n, (ibA + 1) * kTile) + kFwKeys - 1) / kFwKeys;
  const int ntB = hasB ? (min(n, (ibB + 1) * kTile) + kFwKeys - 1) / kFwKeys : 0;
  const int nt = max(ntA, ntB);

  if (threadIdx.x == 0) {
    for (int g = 0; g < 2; ++g) {
      mbar_init(&sh.q_full[g], 1);
      for (int b = 0; b < 2; ++b) {
        mbar_init(&sh.s_full[g][b], 1);
        mbar_init(&sh.p_full[g][b], 4);
      }
      mbar_init(&sh.pv_done[g][0], 1);
      mbar_init(&sh.pv_done[g][1], 1);
      mbar_init(&sh.o_final[g], (g == 0 ? ntA : ntB) >= 2 ? 2 : 1);  // one arrival per issuing warp that has a tile
    }
    for (int i = 0; i < kFwKvSlots; ++i) {
      mbar_init(&sh.kv_full[i], 1);
      mbar_init(&sh.kv_empty[i], G);  // one arrival per group
    }
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, kFwTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;

  // MMA issuer index: (group, tile parity) = (idx % G, idx / G); warps 1..3 and, with two groups, warp 12
  const int mma_idx = (warp >= 1 && warp <= 3) ? warp - 1 : (warp == 12 ? 3 : -1);
  const bool softmax_warp = warp >= 4 && warp < 4 + 4 * G;
  // One branch per register budget (the groups of four warps change theirs right at its top, so that
  // the compiler sees which code runs under which budget).
  if (!softmax_warp) {
  setmaxnreg_dec<kFwRegsIssue>();
  if (warp == 0) {
    // ---------------- TMA producer: Q tiles, then K_0, V_0, K_1, V_1, ... through the slot ring ----
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      for (int g = 0; g < (hasB ? 2 : 1); ++g) {
        unsigned char* dst = q_tiles + g * kTileBytes;
        mbar_expect_tx(&sh.q_full[g], kTileBytes);
        tma_load_tile(dst, &map_q, h, lo + (ibA + g) * kTile, &sh.q_full[g]);
      }
      for (int r = 0; r < 2 * nt; ++r) {
        const int slot = r % kFwKvSlots;
        if (!wait_or_abort(&sh.kv_empty[slot], ((r / kFwKvSlots) & 1) ^ 1, abort_flag)) break;
        const CUtensorMap* map = (r & 1) ? &map_v : &map_k;
        unsigned char* dst = kv_ring + slot * kFwKvSlotBytes;
        const int row0 = lo + (r >> 1) * kFwKeys;
        mbar_expect_tx(&sh.kv_full[slot], kFwKvSlotBytes);
        tma_load_tile(dst, map, h / kv_div, row0, &sh.kv_full[slot]);
      }
    }
  } else if (mma_idx >= 0 && mma_idx < 2 * G) {
    // ---------------- MMA issuers: two warps per softmax group, one for the even key tiles, one for the odd ----
    // A single thread's instruction stream is what bounds the issue of these small matrix instructions: one
    // warp needs about a thousand cycles per action (barrier waits, eight instructions, commits), two
    // actions per tile, while the softmax of a tile takes ~1,300.  So every group has two issuing warps,
    // each with two tile times for its P V(j) and S(j+2); the tensor core takes instructions from all of
    // them.  The whole warp runs the loop (warp-uniform descriptors), one elected lane issues (a single
    // active lane running the loop was slower).
    constexpr uint32_t idesc_s = instr_desc_f16(kTile, kFwKeys, kFmtBF16, kFmtBF16, false, false);
    // V is the MN-major operand.  (Both operands of one instruction must have the same 16-bit format:
    // an fp16 P against a bf16 V is rejected by the hardware as an illegal instruction.)
    constexpr uint32_t idesc_o = instr_desc_f16(kTile, kD, kFmtBF16, kFmtBF16, false, true);
    constexpr int kRing = kFwKvSlots / 2;  // key tiles in the ring: tile j has K in slot 2 (j % kRing), V in the next
    const int g = mma_idx % G, par = mma_idx / G;  // group, parity of this warp's tiles
    const int ntg = g == 0 ? ntA : ntB;
    bool ok = ntg <= par || wait_or_abort(&sh.q_full[g], 0, abort_flag);
    ok = __all_sync(0xffffffffu, ok) != 0;
    if (ok) tc_fence_after();
    const uint32_t q_base = smem_u32(q_tiles + g * kTileBytes);
    const uint32_t sp = tmem + kFwColSP + (uint32_t)g * 128u + (uint32_t)par * 64u;  // this warp's S/P buffer
    const uint32_t d_o = tmem + kFwColO + (uint32_t)g * 128u;
    const uint64_t dq = smem_desc_sw128(q_base, 16, 1024);
    // S_g(js) = Q_g K_js^T into buffer js % 2: needs K_js in shared memory.  The buffer's previous content,
    // P_g(js-2), is read by P V of tile js-2, which this thread issued earlier: the tensor core runs one
    // thread's instructions in order.
    auto issue_s = [&](int js) {
      const int slot = 2 * (js % kRing);
      ok = ok && wait_or_abort(&sh.kv_full[slot], (uint32_t)(js / kRing) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok) != 0;
      if (!ok) return;
      tc_fence_after();
      FWD_TL(g, js, 5);
      // descriptors once per tile; a K step only moves the start-address field of the low word
      const uint64_t dk = smem_desc_sw128(smem_u32(kv_ring + slot * kFwKvSlotBytes), 16, 1024);
      if (elect_one()) {
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t qoff = (uint32_t)(ks >> 2) * kBoxBytes + (uint32_t)(ks & 3) * 32u;
          const uint32_t koff = (uint32_t)(ks >> 2) * (kFwKvSlotBytes / 2) + (uint32_t)(ks & 3) * 32u;
          if (ks == 0)
            mma_ss_lohi<false>(sp, desc_lo(dq), desc_hi(dq), desc_lo(dk), desc_hi(dk), idesc_s);
          else
            mma_ss_lohi<true>(sp, desc_lo(dq) + (qoff >> 4), desc_hi(dq), desc_lo(dk) + (koff >> 4), desc_hi(dk), idesc_s);
        }
        mma_commit(&sh.s_full[g][par]);
        FWD_TL(g, js, 0);
        mma_commit(&sh.kv_empty[slot]);  // K_js may be refilled once every group's scores have read it
      }
      __syncwarp();
    };
    if (par < ntg) issue_s(par);
    for (int j = par; j < ntg && ok; j += 2) {
      // ---- O_g += P_g(j) V_j: needs P_g(j) in tensor memory and V_j in shared memory ----
      const int slot = 2 * (j % kRing) + 1;
      FWD_TL(g, j, 6);
      // The products of a group accumulate into O_g in tile order: this one is issued when the previous
      // tile's (the other warp's) is complete.  That fixes the order of the fp32 additions, so every bit of
      // the output is the same in every run, and keeps P V(0), which initialises O_g, first.  (In steady
      // state that product completed a tile time ago: the wait costs its own latency only.)
      if (j >= 1) ok = ok && wait_or_abort(&sh.pv_done[g][par ^ 1], (uint32_t)((j - 1) >> 1) & 1u, abort_flag);
      ok = ok && wait_or_abort(&sh.p_full[g][par], (uint32_t)(j >> 1) & 1u, abort_flag);
      FWD_TL(g, j, 7);
      ok = ok && wait_or_abort(&sh.kv_full[slot], (uint32_t)(j / kRing) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok) != 0;
      if (!ok) break;
      tc_fence_after();
      FWD_TL(g, j, 2);
      const uint64_t dv = smem_desc_sw128(smem_u32(kv_ring + slot * kFwKvSlotBytes), kFwKvSlotBytes / 2, 1024);
      const volatile uint32_t* ln = sh.lo_need[g][par];  // (tile j uses buffer j % 2 == par)
      const bool need_lo = kFwSplitP && (ln[0] | ln[1] | ln[2] | ln[3]) != 0u;
      if (elect_one()) {
        if (j == 0) mma_ts_lohi<false>(d_o, sp, desc_lo(dv), desc_hi(dv), idesc_o);
        else mma_ts_lohi<true>(d_o, sp, desc_lo(dv), desc_hi(dv), idesc_o);
#pragma unroll
        for (int ks = 1; ks < kFwKeys / 16; ++ks)  // hi columns
          mma_ts_lohi<true>(d_o, sp + (uint32_t)ks * 8u, desc_lo(dv) + (((uint32_t)ks * 2048u) >> 4), desc_hi(dv), idesc_o);
        if (need_lo) {
#pragma unroll
          for (int ks = 0; ks < kFwKeys / 16; ++ks)  // lo columns, same V rows
            mma_ts_lohi<true>(d_o, sp + 32u + (uint32_t)ks * 8u, desc_lo(dv) + (((uint32_t)ks * 2048u) >> 4), desc_hi(dv), idesc_o);
        }
        FWD_TL(g, j, 8);
        mma_commit(&sh.pv_done[g][par]);
        if (j + 2 >= ntg) mma_commit(&sh.o_final[g]);  // this warp's last tile
        FWD_TL(g, j, 4);
        mma_commit(&sh.kv_empty[slot]);
        FWD_TL(g, j, 9);
      }
      __syncwarp();
      if (j + 2 < ntg) issue_s(j + 2);
    }
    // Tiles of this parity that the group never uses (its query block ends earlier, or it does not exist):
    // the ring still expects one arrival per group and slot, given here as soon as the tile has landed.
    for (int j = ntg + ((ntg ^ par) & 1); j < nt && ok; j += 2) {
      const int slot = 2 * (j % kRing);
      const uint32_t ph = (uint32_t)(j / kRing) & 1u;
      ok = wait_or_abort(&sh.kv_full[slot], ph, abort_flag);
      if (ok && lane == 0) mbar_arrive(&sh.kv_empty[slot]);
      ok = ok && wait_or_abort(&sh.kv_full[slot + 1], ph, abort_flag);
      if (ok && lane == 0) mbar_arrive(&sh.kv_empty[slot + 1]);
      ok = __all_sync(0xffffffffu, ok) != 0;
    }
  }
  } else {
    setmaxnreg_inc<kFwRegsSoftmax>();
    // ---------------- softmax groups: one thread per query row ----------------
    const int g = (warp - 4) >> 2;             // 0: group A, 1: group B
    const int ib = g == 0 ? ibA : ibB;
    const int ntg = g == 0 ? ntA : ntB;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int qi = ib * kTile + row;           // query position inside the sequence
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t tmem_o = tmem + kFwColO + (uint32_t)g * 128u + lane_addr;
    const uint32_t tmem_sp = tmem + kFwColSP + (uint32_t)g * 128u + lane_addr;  // + 64 (j & 1)
    bool ok = true;
    float m_used = -INFINITY;
    float2 l2 = make_float2(0.f, 0.f);  // row sum, even and odd keys apart (packed fp32x2 adds)
#ifdef H2O_PHASE_TIMERS
    long long prof_[5] = {0, 0, 0, 0, 0};
#endif
    for (int j = 0; j < ntg && ok; ++j) {
      FWD_CLK(c0_);
      ok = __all_sync(0xffffffffu, wait_or_abort(&sh.s_full[g][j & 1], (uint32_t)(j >> 1) & 1u, abort_flag));  // collectives below
      if (!ok) break;
      tc_fence_after();
      FWD_CLK(c1_);
      FWD_TL(g, j, 1);
      const uint32_t buf = tmem_sp + (uint32_t)(j & 1) * 64u;
      uint32_t r0[32], r1[32];
      tmem_ld32(buf, r0);
      tmem_ld32(buf + 32u, r1);
      tmem_wait_ld();
      FWD_CLK(c2_);
      const int key0 = j * kFwKeys;
      const bool masked_tile = key0 + kFwKeys - 1 > ib * kTile;  // tile reaches past this block's first query
      // raw scores stay unscaled: the scale is positive, so the maximum commutes with it and the
      // multiplication is folded into the exponent's fused multiply-add below
      if (masked_tile) {
#pragma unroll
        for (int c2 = 0; c2 < kFwKeys; ++c2)
          if (key0 + c2 > qi) (c2 < 32 ? r0[c2] : r1[c2 - 32]) = 0xff800000u;  // -inf, causal: key <= query
      }
      float m_raw = -INFINITY;
#pragma unroll
      for (int c2 = 0; c2 < kFwKeys; c2 += 2)  // three-input maximum: half the instructions on the ALU pipe
        m_raw = max3(m_raw, __uint_as_float(c2 < 32 ? r0[c2] : r1[c2 - 32]),
                     __uint_as_float(c2 < 32 ? r0[c2 + 1] : r1[c2 - 31]));
      const float m_tile = m_raw * scale2;
      const bool need = m_tile > m_used + kRescaleThreshold;
      if (j == 0) {
        m_used = m_tile;  // key 0 is visible to every row, so this is finite
      } else {
        const bool rescale = __any_sync(0xffffffffu, need);
        if (rescale) {
          // O_g must include tile j-1 before it is rescaled (P V of tile j is issued only after this
          // tile's probabilities, so it sees the rescaled rows)
          ok = __all_sync(0xffffffffu, wait_or_abort(&sh.pv_done[g][(j - 1) & 1], (uint32_t)((j - 1) >> 1) & 1u, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const float m_new = need ? m_tile : m_used;
          const float alpha = ex2(m_used - m_new);
          l2 = __fmul2_rn(l2, make_float2(alpha, alpha));
          m_used = m_new;
#pragma unroll
          for (int cc = 0; cc < kD / 32; ++cc) {
            uint32_t o[32];
            tmem_ld32(tmem_o + (uint32_t)cc * 32u, o);
            tmem_wait_ld();
#pragma unroll
            for (int c2 = 0; c2 < 32; ++c2) o[c2] = __float_as_uint(__uint_as_float(o[c2]) * alpha);
            tmem_st32(tmem_o + (uint32_t)cc * 32u, o);
          }
          tmem_wait_st();
        }
      }
      const float neg_m = -m_used;
      FWD_CLK(c3_);
      // probabilities relative to the reference maximum as bf16 hi (columns 0..31) and bf16 lo
      // (columns 32..63): column c holds keys 2c and 2c+1
      uint32_t hw[32];
      [[maybe_unused]] uint32_t lw[32];
      float p_max = 0.f;
#pragma unroll
      for (int c = 0; c < 32; ++c) {
        const float s0 = __uint_as_float(c < 16 ? r0[2 * c] : r1[2 * c - 32]);
        const float s1 = __uint_as_float(c < 16 ? r0[2 * c + 1] : r1[2 * c - 31]);
        const float2 x = __ffma2_rn(make_float2(s0, s1), make_float2(scale2, scale2), make_float2(neg_m, neg_m));
        const float2 pp = make_float2(ex2(x.x), ex2(x.y));
        l2 = __fadd2_rn(l2, pp);
        p_max = max3(p_max, pp.x, pp.y);
        const __nv_bfloat162 hi2 = __floats2bfloat162_rn(pp.x, pp.y);
        hw[c] = *reinterpret_cast<const uint32_t*>(&hi2);
        if constexpr (kFwSplitP) {
          const float2 lo = __ffma2_rn(__bfloat1622float2(hi2), make_float2(-1.f, -1.f), pp);  // exact remainder
          lw[c] = Vec16<__nv_bfloat16>::pack2(lo.x, lo.y);
        }
      }
      tmem_st32(buf, hw);        // over the scores, which are in registers by now
      if constexpr (kFwSplitP) tmem_st32(buf + 32u, lw);
      tmem_wait_st();
      FWD_CLK(c4_);
      FWD_TL(g, j, 3);
      tc_fence_before();
      const bool lo_vote = __any_sync(0xffffffffu, p_max > kFwLoThreshold * (l2.x + l2.y));
      if (lane == 0) {
        sh.lo_need[g][j & 1][quarter] = lo_vote ? 1u : 0u;
        mbar_arrive(&sh.p_full[g][j & 1]);
      }
      FWD_ADD(0, c0_, c1_);
      FWD_ADD(1, c1_, c2_);
      FWD_ADD(2, c2_, c3_);
      FWD_ADD(3, c3_, c4_);
    }
#ifdef H2O_PHASE_TIMERS
    if (lane == 0 && quarter == 0) {
      for (int i = 0; i < 4; ++i) atomicAdd(&g_fwd_prof[i], (unsigned long long)prof_[i]);
      atomicAdd(&g_fwd_prof[5], (unsigned long long)ntg);
    }
#endif
    if (ntg > 0) {
      if (ok) ok = __all_sync(0xffffffffu, wait_or_abort(&sh.o_final[g], 0, abort_flag));
      if (ok) {
        tc_fence_after();
        const float inv_l = 1.0f / (l2.x + l2.y);
        __nv_bfloat16* orow = out + ((int64_t)(lo + qi) * n_heads + h) * kD;
#pragma unroll
        for (int cc = 0; cc < kD / 32; ++cc) {
          uint32_t o[32];
          tmem_ld32(tmem_o + (uint32_t)cc * 32u, o);
          tmem_wait_ld();
          if (qi < n) store_out_32(orow + cc * 32, o, inv_l, wide_out);
        }
        if (qi < n) s.rowstat[(int64_t)h * s.total_tokens + lo + qi] = make_float2(m_used, inv_l);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(status, 0, H2O_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kFwTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Forward for prompts of up to kFwShortPrompt tokens: persistent blocks, one softmax group, two blocks per SM
// ---------------------------------------------------------------------------------------------
// Same arithmetic, tiles and tensor-memory layout as the one-group instance of the kernel above, but a
// block walks over work items (unit, query block) instead of ending after one: barriers, tensor memory
// and the K/V ring stay up, so an item's first loads and score tiles overlap the previous item's last
// tiles and its output.  With 512-token prompts a block of the kernel above spends more time on its fixed
// cost (allocation, first loads, pipeline fill, output, exit and relaunch) than on its five tiles; with
// 2048-token prompts that cost is still a quarter of a block's time.
// All counters run over the block's whole sequence of key tiles: tile T uses ring slots 2 (T % 2) and
// + 1, score buffer T % 2 and the issuing warp T % 2; a warp issues P V(T), then S(T + 2), which may
// belong to the next item.
constexpr int kFsThreads = 256;  // warp 0 TMA, warps 1, 2 MMA (even, odd tiles), warp 3 idle, warps 4..7 softmax
constexpr int kFsKvSlots = 4;
constexpr int kFsDescs = 8;
constexpr uint32_t kFsTmemCols = 256;  // O 128 columns, two score / probability buffers of 64
// register budgets after the block's start with 128 per thread (the issuers keep two tile walkers)
constexpr int kFsRegsIssue = 88, kFsRegsSoftmax = 168;

struct FsShared {
  uint64_t q_full, q_empty;  // Q of the item is in shared memory / both issuing warps are done with it
  uint64_t kv_full[kFsKvSlots], kv_empty[kFsKvSlots];
  uint64_t s_full[2], p_full[2], pv_done[2];
  uint64_t o_final;          // both issuing warps' last products of the item are complete
  uint32_t tmem_base;
  int abort_flag;
  uint32_t lo_need[2][4];    // [buffer][softmax warp], as in FwShared
  // The producer thread alone looks items up (two dependent loads and divisions per item); it leaves each
  // item's description here before it loads the item's Q.  The S walkers wait for q_full of every item
  // in order and read entry ic % 8 then; the same threads' P V walkers come later; the softmax warps read
  // it after they have seen the item's first score tile (issued behind that wait).  `last` ends the walk;
  // a block without items gets nt == 0 in entry 0.  `start` (used once) tells the softmax warps that
  // entry 0 is there.  (The producer is never more than three items ahead of the slowest reader: Q of
  // item ic+1 waits for the last scores of item ic.)
  uint64_t start;
  struct Desc {
    int h, lo, n, ib, nt, last;
  } desc[kFsDescs];
};

struct FsItem {
  int h, lo, n;  // head, first token and length of the sequence
  int ib, nt;    // query block, key tiles
};
// Item order: units in groups of `grp` (small enough for their K and V to stay in L2 while the group is
// being worked on); inside a group every unit's longest query block first, then every unit's second
// longest, ...: long items start early, the ones claimed last are short.
struct FsOrder {
  int n_heads, units, grp, n_groups, n_items;  // heads and units of the QUERY side
  int kv_div;                                  // query heads per K/V head
  const int32_t* item_base;  // [n_groups + 1] first item index of every group (host-built from the prompt lengths:
                             // a group has as many levels x as its longest sequence has query blocks, so that
                             // a ragged batch does not make most indices name blocks that do not exist)
};
// g: group of the previous item this thread looked up (item indices only grow)
__device__ __forceinline__ bool fs_item(const PrefillScratch& s, const FsOrder& o, int w, int& g, FsItem& it) {
  while (g + 1 < o.n_groups && w >= o.item_base[g + 1]) ++g;
  const int r = w - o.item_base[g];
  const int in_group = min(o.grp, o.units - g * o.grp);
  const int x = r / in_group, uu = r - x * in_group;
  const int u = g * o.grp + uu;
  const int seq = u / o.n_heads;
  it.h = u - seq * o.n_heads;
  it.lo = s.cu[seq];
  it.n = s.cu[seq + 1] - it.lo;
  const int nb = (it.n + kTile - 1) / kTile;
  if (x >= nb) return false;  // a shorter sequence of the group
  it.ib = nb - 1 - x;
  it.nt = (min(it.n, (it.ib + 1) * kTile) + kFwKeys - 1) / kFwKeys;  // keys 0 .. min(n, (ib+1)*128) - 1
  return true;
}

__global__ void __launch_bounds__(kFsThreads, 2)
fwd_tc_short_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, PrefillScratch s, FsOrder order, float scale2,
                    __nv_bfloat16* __restrict__ out, int32_t* status) {
  const int n_heads = order.n_heads, n_items = order.n_items;
  extern __shared__ unsigned char dyn_raw[];
  __shared__ FsShared sh;
  const bool wide_out = (reinterpret_cast<uintptr_t>(out) & 31u) == 0;
  unsigned char* dyn = dyn_raw + ((1024u - (smem_u32(dyn_raw) & 1023u)) & 1023u);
  unsigned char* q_tile = dyn;                // 32 KB
  unsigned char* kv_ring = dyn + kTileBytes;  // four slots of 16 KB
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#ifdef H2O_PHASE_TIMERS
  const bool tl_on_ = blockIdx.x == 0 && lane == 0 && (warp == 1 || warp == 2 || warp == 4);
#endif

  if (threadIdx.x == 0) {
    mbar_init(&sh.q_full, 1);
    mbar_init(&sh.q_empty, 2);
    for (int i = 0; i < kFsKvSlots; ++i) {
      mbar_init(&sh.kv_full[i], 1);
      mbar_init(&sh.kv_empty[i], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sh.s_full[b], 1);
      mbar_init(&sh.p_full[b], 4);
      mbar_init(&sh.pv_done[b], 1);
    }
    mbar_init(&sh.o_final, 2);
    mbar_init(&sh.start, 1);
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, kFsTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;
  const bool softmax_warp = warp >= 4;

  // One branch per register budget (the groups of four warps change theirs right at its top, so that
  // the compiler sees which code runs under which budget).
  if (!softmax_warp) {
  setmaxnreg_dec<kFsRegsIssue>();
  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      // Items are claimed from a counter in the order of the item index (unit by unit, a unit's longest
      // query block first): blocks that finish early take more, and the items of a unit run close together
      // in time, so its K and V are read from memory once.  The claim (an atomic and two dependent loads)
      // is made two items ahead: `last` of an item needs to know whether another one follows, and the
      // lookup must not sit between an item's end and the next one's first loads.
      int g_at = 0;
      auto claim = [&](FsItem& it) {  // next existing item; n_items: none left
        int w;
        do {
          w = atomicAdd(s.work, 1);
        } while (w < n_items && !fs_item(s, order, w, g_at, it));
        return w < n_items ? w : n_items;
      };
      FsItem it, nx, nx2;
      int w = claim(it);
      int wn = w < n_items ? claim(nx) : n_items;
      bool ok = true;
      if (w >= n_items) {  // nothing for this block
        sh.desc[0].nt = 0;
        sh.desc[0].last = 1;
        mbar_arrive(&sh.start);
        mbar_arrive(&sh.q_full);
      }
      for (int ic = 0, T = 0; ok && w < n_items; ++ic) {
        int wn2 = n_items;
        // the item's Q tile, once both issuing warps are done with the previous one
        if (ic >= 1) ok = wait_or_abort(&sh.q_empty, (uint32_t)(ic - 1) & 1u, abort_flag);
        if (!ok) break;
        FsShared::Desc& d = sh.desc[ic % kFsDescs];
        d.h = it.h;
        d.lo = it.lo;
        d.n = it.n;
        d.ib = it.ib;
        d.nt = it.nt;
        d.last = wn >= n_items;
        if (ic == 0) mbar_arrive(&sh.start);
        mbar_expect_tx(&sh.q_full, kTileBytes);  // (release: the description is written before)
        tma_load_tile(q_tile, &map_q, it.h, it.lo + it.ib * kTile, &sh.q_full);
        for (int j = 0; j < it.nt && ok; ++j, ++T) {
          const int slot = 2 * (T & 1);
          const uint32_t par = ((uint32_t)(T >> 1) & 1u) ^ 1u;
          const int row0 = it.lo + j * kFwKeys;
#pragma unroll
          for (int r = 0; r < 2 && ok; ++r) {
            ok = wait_or_abort(&sh.kv_empty[slot + r], par, abort_flag);
            if (!ok) break;
            const CUtensorMap* map = r ? &map_v : &map_k;
            unsigned char* dst = kv_ring + (slot + r) * kFwKvSlotBytes;
            mbar_expect_tx(&sh.kv_full[slot + r], kFwKvSlotBytes);
            tma_load_tile(dst, map, it.h / order.kv_div, row0, &sh.kv_full[slot + r]);
          }
          // the ring is full after the item's first tiles: time for the lookup two items ahead
          if (j == min(1, it.nt - 1) && wn < n_items) wn2 = claim(nx2);
        }
        w = wn;
        it = nx;
        wn = wn2;
        nx = nx2;
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ---------------- MMA issuers: warp 1 the even key tiles, warp 2 the odd ones ----------------
    constexpr uint32_t idesc_s = instr_desc_f16(kTile, kFwKeys, kFmtBF16, kFmtBF16, false, false);
    constexpr uint32_t idesc_o = instr_desc_f16(kTile, kD, kFmtBF16, kFmtBF16, false, true);
    const int par = warp - 1;
    const uint32_t sp = tmem + 128u + (uint32_t)par * 64u;  // this warp's score / probability buffer
    const uint32_t d_o = tmem;
    const uint64_t dq = smem_desc_sw128(smem_u32(q_tile), 16, 1024);
    bool ok = true;
    // This warp's tiles are T = par, par + 2, ...  It needs only the position inside the item (first,
    // second, last own tile) and the item count; items in which it has no tile (a single tile, of the
    // other parity) still get its arrival on the per-item barriers (q_empty from the S walker, o_final
    // from the P V walker).
    struct Lean {
      int j, T, ic, nt, last;
    };
    // enter item k.ic: the S walker waits for its Q (and with it for its description), the P V walker of
    // the same thread comes later; false for a block without items
    auto lean_enter = [&](Lean& k, bool wait_q) {
      if (wait_q) ok = ok && wait_or_abort(&sh.q_full, (uint32_t)k.ic & 1u, abort_flag);
      if (!ok) return false;
      const volatile FsShared::Desc& d = sh.desc[k.ic % kFsDescs];
      k.nt = d.nt;
      k.last = d.last;
      return k.nt > 0;
    };
    auto lean_first = [&](Lean& k, bool wait_q) {
      k.j = k.T = k.ic = 0;
      return lean_enter(k, wait_q);
    };
    auto lean_next = [&](Lean& k, bool wait_q) {
      ++k.T;
      if (++k.j < k.nt) return true;
      if (k.last) return false;
      k.j = 0;
      ++k.ic;
      return lean_enter(k, wait_q);
    };
    // from a tile of the other parity (an item of one tile gets the direct arrival) to the next own tile
    auto skip_other = [&](Lean& k, bool& have, uint64_t* item_bar, bool wait_q) {
      if (k.nt == 1 && lane == 0) mbar_arrive(item_bar);
      have = lean_next(k, wait_q);
    };
    Lean ks_, kp_;
    bool have_s = lean_first(ks_, true);
    if (have_s && par == 1) skip_other(ks_, have_s, &sh.q_empty, true);
    bool have_p = lean_first(kp_, false);
    if (have_p && par == 1) skip_other(kp_, have_p, &sh.o_final, false);
    // The S walker runs one own tile ahead of the P V walker: S(T + 2) is issued right behind P V(T) by
    // the same thread, and its buffer is the one that product reads (the tensor core runs one thread's
    // instructions in order).
    // Both walkers move on at the START of their next step.  For the S walker this keeps the wait for the
    // next item's Q behind the product that may be ready; the P V walker then enters an item only after the
    // S walker has (it reads the item's description without a wait of its own).
    bool s_advance = false, p_advance = false;
    for (bool first = true; ok; first = false) {
      if (!first) {
        if (p_advance) {
          have_p = lean_next(kp_, false);
          if (have_p) skip_other(kp_, have_p, &sh.o_final, false);
          p_advance = false;
        }
        if (!have_p) break;
        // ---- O += P(T) V_T ----
        const int T = kp_.T, j = kp_.j;
        const int slot = 2 * (T & 1) + 1;
        // The products of one item accumulate into O in tile order: this one is issued when the previous
        // tile's (the other warp's) is complete.  That fixes the order of the fp32 additions, so every bit
        // of the output is the same in every run, and keeps the first product, which initialises O, first.
        // (In steady state that product completed a tile time ago: the wait costs its own latency only.)
        if (j >= 1) ok = ok && wait_or_abort(&sh.pv_done[par ^ 1], (uint32_t)((T - 1) >> 1) & 1u, abort_flag);
        ok = ok && wait_or_abort(&sh.p_full[par], (uint32_t)(T >> 1) & 1u, abort_flag);
        ok = ok && wait_or_abort(&sh.kv_full[slot], (uint32_t)(T >> 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok) != 0;
        if (!ok) break;
        tc_fence_after();
        FWD_TL(0, T, 2);
        const uint64_t dv = smem_desc_sw128(smem_u32(kv_ring + slot * kFwKvSlotBytes), kFwKvSlotBytes / 2, 1024);
        const volatile uint32_t* ln = sh.lo_need[par];  // (tile T uses buffer T % 2 == par)
        const bool need_lo = kFwSplitP && (ln[0] | ln[1] | ln[2] | ln[3]) != 0u;
        if (elect_one()) {
          // (P(0) of an item is stored only after the softmax warps have read the previous item's O)
          if (j == 0) mma_ts_lohi<false>(d_o, sp, desc_lo(dv), desc_hi(dv), idesc_o);
          else mma_ts_lohi<true>(d_o, sp, desc_lo(dv), desc_hi(dv), idesc_o);
#pragma unroll
          for (int ks = 1; ks < kFwKeys / 16; ++ks)  // hi columns
            mma_ts_lohi<true>(d_o, sp + (uint32_t)ks * 8u, desc_lo(dv) + (((uint32_t)ks * 2048u) >> 4), desc_hi(dv), idesc_o);
          if (need_lo) {
#pragma unroll
            for (int ks = 0; ks < kFwKeys / 16; ++ks)  // lo columns, same V rows
              mma_ts_lohi<true>(d_o, sp + 32u + (uint32_t)ks * 8u, desc_lo(dv) + (((uint32_t)ks * 2048u) >> 4), desc_hi(dv), idesc_o);
          }
          mma_commit(&sh.pv_done[par]);
          if (j + 2 >= kp_.nt) mma_commit(&sh.o_final);  // this warp's last product of the item
          mma_commit(&sh.kv_empty[slot]);
          FWD_TL(0, T, 4);
        }
        __syncwarp();
        p_advance = true;
      }
      if (s_advance) {
        // (only now, behind the product above: entering the next item waits for its Q, and a product that
        //  is ready must not wait behind that)
        have_s = lean_next(ks_, true);
        if (have_s) skip_other(ks_, have_s, &sh.q_empty, true);
        s_advance = false;
      }
      if (have_s) {
        // ---- S(T) = Q K_T^T ----
        const int T = ks_.T;
        const int slot = 2 * (T & 1);
        ok = ok && wait_or_abort(&sh.kv_full[slot], (uint32_t)(T >> 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok) != 0;
        if (!ok) break;
        tc_fence_after();
        FWD_TL(0, T, 5);
        const uint64_t dk = smem_desc_sw128(smem_u32(kv_ring + slot * kFwKvSlotBytes), 16, 1024);
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks) {
            const uint32_t qoff = (uint32_t)(ks >> 2) * kBoxBytes + (uint32_t)(ks & 3) * 32u;
            const uint32_t koff = (uint32_t)(ks >> 2) * (kFwKvSlotBytes / 2) + (uint32_t)(ks & 3) * 32u;
            if (ks == 0)
              mma_ss_lohi<false>(sp, desc_lo(dq), desc_hi(dq), desc_lo(dk), desc_hi(dk), idesc_s);
            else
              mma_ss_lohi<true>(sp, desc_lo(dq) + (qoff >> 4), desc_hi(dq), desc_lo(dk) + (koff >> 4), desc_hi(dk), idesc_s);
          }
          mma_commit(&sh.s_full[par]);
          mma_commit(&sh.kv_empty[slot]);
          if (ks_.j + 2 >= ks_.nt) mma_commit(&sh.q_empty);  // this warp's last score tile of the item
          FWD_TL(0, T, 0);
        }
        __syncwarp();
        s_advance = true;
      } else if (first) {
        break;
      }
    }
  }
  } else {
    setmaxnreg_inc<kFsRegsSoftmax>();
    // ---------------- softmax: one thread per query row ----------------
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t tmem_o = tmem + lane_addr;
    const uint32_t tmem_sp = tmem + 128u + lane_addr;  // + 64 (T & 1)
    bool ok = true;
    float m_used = -INFINITY;
    float2 l2 = make_float2(0.f, 0.f);  // row sum, even and odd keys apart (packed fp32x2 adds)
    FsItem it;
    int T = 0;  // key tiles so far, over all items
    ok = __all_sync(0xffffffffu, wait_or_abort(&sh.start, 0, abort_flag));  // entry 0 of the descriptions is there
    for (int ic = 0, last = 0; ok && !last; ++ic) {
      // the item's description: readable once the item's first score tile has been seen
      bool first_seen = false;
      if (ic > 0) {
        ok = __all_sync(0xffffffffu, wait_or_abort(&sh.s_full[T & 1], (uint32_t)(T >> 1) & 1u, abort_flag));
        if (!ok) break;
        first_seen = true;
      }
      {
        const volatile FsShared::Desc& d = sh.desc[ic % kFsDescs];
        it.h = d.h;
        it.lo = d.lo;
        it.n = d.n;
        it.ib = d.ib;
        it.nt = d.nt;
        last = d.last;
      }
      if (it.nt == 0) break;
      const int qi = it.ib * kTile + row;  // query position inside the sequence
      for (int j = 0; j < it.nt && ok; ++j, ++T) {
      if (!(j == 0 && first_seen))
        ok = __all_sync(0xffffffffu, wait_or_abort(&sh.s_full[T & 1], (uint32_t)(T >> 1) & 1u, abort_flag));  // collectives below
      if (!ok) break;
      tc_fence_after();
      FWD_TL(0, T, 1);
      const uint32_t buf = tmem_sp + (uint32_t)(T & 1) * 64u;
      uint32_t r0[32], r1[32];
      tmem_ld32(buf, r0);
      tmem_ld32(buf + 32u, r1);
      tmem_wait_ld();
      const int key0 = j * kFwKeys;
      const bool masked_tile = key0 + kFwKeys - 1 > it.ib * kTile;  // tile reaches past this block's first query
      if (masked_tile) {
#pragma unroll
        for (int c2 = 0; c2 < kFwKeys; ++c2)
          if (key0 + c2 > qi) (c2 < 32 ? r0[c2] : r1[c2 - 32]) = 0xff800000u;  // -inf, causal: key <= query
      }
      float m_raw = -INFINITY;
#pragma unroll
      for (int c2 = 0; c2 < kFwKeys; c2 += 2)
        m_raw = max3(m_raw, __uint_as_float(c2 < 32 ? r0[c2] : r1[c2 - 32]),
                     __uint_as_float(c2 < 32 ? r0[c2 + 1] : r1[c2 - 31]));
      const float m_tile = m_raw * scale2;
      const bool need = m_tile > m_used + kRescaleThreshold;
      if (j == 0) {
        m_used = m_tile;  // key 0 is visible to every row, so this is finite
        l2 = make_float2(0.f, 0.f);
      } else {
        const bool rescale = __any_sync(0xffffffffu, need);
        if (rescale) {
          // O must include tile T-1 before it is rescaled
          ok = __all_sync(0xffffffffu, wait_or_abort(&sh.pv_done[(T - 1) & 1], (uint32_t)((T - 1) >> 1) & 1u, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const float m_new = need ? m_tile : m_used;
          const float alpha = ex2(m_used - m_new);
          l2 = __fmul2_rn(l2, make_float2(alpha, alpha));
          m_used = m_new;
#pragma unroll
          for (int cc = 0; cc < kD / 32; ++cc) {
            uint32_t o[32];
            tmem_ld32(tmem_o + (uint32_t)cc * 32u, o);
            tmem_wait_ld();
#pragma unroll
            for (int c2 = 0; c2 < 32; ++c2) o[c2] = __float_as_uint(__uint_as_float(o[c2]) * alpha);
            tmem_st32(tmem_o + (uint32_t)cc * 32u, o);
          }
          tmem_wait_st();
        }
      }
      const float neg_m = -m_used;
      uint32_t hw[32];
      [[maybe_unused]] uint32_t lw[32];
      float p_max = 0.f;
#pragma unroll
      for (int c = 0; c < 32; ++c) {
        const float s0 = __uint_as_float(c < 16 ? r0[2 * c] : r1[2 * c - 32]);
        const float s1 = __uint_as_float(c < 16 ? r0[2 * c + 1] : r1[2 * c - 31]);
        const float2 x = __ffma2_rn(make_float2(s0, s1), make_float2(scale2, scale2), make_float2(neg_m, neg_m));
        const float2 pp = make_float2(ex2(x.x), ex2(x.y));
        l2 = __fadd2_rn(l2, pp);
        p_max = max3(p_max, pp.x, pp.y);
        const __nv_bfloat162 hi2 = __floats2bfloat162_rn(pp.x, pp.y);
        hw[c] = *reinterpret_cast<const uint32_t*>(&hi2);
        if constexpr (kFwSplitP) {
          const float2 lo = __ffma2_rn(__bfloat1622float2(hi2), make_float2(-1.f, -1.f), pp);  // exact remainder
          lw[c] = Vec16<__nv_bfloat16>::pack2(lo.x, lo.y);
        }
      }
      tmem_st32(buf, hw);  // over the scores, which are in registers by now
      if constexpr (kFwSplitP) tmem_st32(buf + 32u, lw);
      tmem_wait_st();
      tc_fence_before();
      const bool lo_vote = __any_sync(0xffffffffu, p_max > kFwLoThreshold * (l2.x + l2.y));
      if (lane == 0) {
        sh.lo_need[T & 1][quarter] = lo_vote ? 1u : 0u;
        mbar_arrive(&sh.p_full[T & 1]);
      }
      FWD_TL(0, T, 3);
      }
      if (ok) {  // the item's output
        ok = __all_sync(0xffffffffu, wait_or_abort(&sh.o_final, (uint32_t)ic & 1u, abort_flag));
        if (!ok) break;
        tc_fence_after();
        FWD_TL(0, T - 1, 6);
        const float inv_l = 1.0f / (l2.x + l2.y);
        __nv_bfloat16* orow = out + ((int64_t)(it.lo + qi) * n_heads + it.h) * kD;
#pragma unroll
        for (int cc = 0; cc < kD / 32; ++cc) {
          uint32_t o[32];
          tmem_ld32(tmem_o + (uint32_t)cc * 32u, o);
          tmem_wait_ld();
          if (qi < it.n) store_out_32(orow + cc * 32, o, inv_l, wide_out);
        }
        if (qi < it.n) s.rowstat[(int64_t)it.h * s.total_tokens + it.lo + qi] = make_float2(m_used, inv_l);
        // (the next item's first probabilities, which release its first P V and with it the overwrite
        //  of O, are stored by these same warps after this point)
        tc_fence_before();
        FWD_TL(0, T - 1, 7);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && sh.abort_flag) atomicCAS(status, 0, H2O_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kFsTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Tensor maps
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Softmax scale times log2(e), rounded once.  The forward and the column-sum kernel use the same
// value, so a row's probabilities sum to one exactly as the forward pass normalised them.
float make_scale2(float c) { return (float)((double)c * kLog2eD); }

}  // namespace

// [total_tokens, n_heads, 128] bf16, box = rows x 1 head x 64 elements (128 bytes), 128-byte swizzle
// [total_tokens, n_heads, 128] bf16 as {64 elements, tokens, 2 halves, heads}: one box = rows x both halves
// of one head, 128-byte swizzle, landing as [half][row][128 bytes]
bool make_whole_tile_map(CUtensorMap* map, const void* base, int64_t total_tokens, int n_heads, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {64, (cuuint64_t)total_tokens, 2, (cuuint64_t)n_heads};
  const cuuint64_t strides[3] = {(cuuint64_t)n_heads * kD * 2, 128, (cuuint64_t)kD * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 2, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tile_map(CUtensorMap* map, const void* base, int64_t total_tokens, int n_heads, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)n_heads, (cuuint64_t)total_tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)n_heads * kD * 2};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

#ifdef H2O_PHASE_TIMERS
extern "C" int h2o_debug_fwd_timeline(long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_fwd_tl, sizeof(g_fwd_tl));
}
extern "C" int h2o_debug_fwd_prof(unsigned long long* host, int reset) {
  if (reset) {
    unsigned long long z[8] = {};
    return (int)cudaMemcpyToSymbol(g_fwd_prof, z, sizeof(z));
  }
  return (int)cudaMemcpyFromSymbol(host, g_fwd_prof, sizeof(unsigned long long) * 8);
}
#endif

namespace {

template <int G>
cudaError_t launch_fwd_g(const CUtensorMap& map_q, const CUtensorMap& map_k, const CUtensorMap& map_v, const CacheView& c,
                         const PrefillScratch& s, int max_seqlen, void* out, cudaStream_t stream) {
  const int smem = G * kTileBytes + fw_kv_slots(G) * kFwKvSlotBytes + 1024;
  static unsigned long long attr_flags = 0;  // one word per template instance, one bit per device
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(fwd_tc_kernel<G>), smem, &attr_flags);
    if (e != cudaSuccess) return e;
  }
  const int nb = (max_seqlen + kTile - 1) / kTile;
  dim3 grid((unsigned)(G == 2 ? (nb + 1) / 2 : nb), (unsigned)(c.units * c.group));
  fwd_tc_kernel<G><<<grid, fw_threads(G), smem, stream>>>(map_q, map_k, map_v, s, c.n_heads * c.group, c.group,
                                                         make_scale2(c.scale), static_cast<__nv_bfloat16*>(out), c.status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_tc(const CacheView& c, const PrefillScratch& s, int max_seqlen, const void* q, const void* k,
                          const void* v, void* out, cudaStream_t stream) {
  CUtensorMap map_q, map_k, map_v;
  if (!make_whole_tile_map(&map_q, q, s.total_tokens, c.n_heads * c.group, kTile) ||
      !make_whole_tile_map(&map_k, k, s.total_tokens, c.n_heads, kFwKeys) ||
      !make_whole_tile_map(&map_v, v, s.total_tokens, c.n_heads, kFwKeys))
    return cudaErrorInvalidValue;
  // short prompts: one query block per thread block, two blocks per SM; long ones: two query blocks share
  // every K/V tile
  if (max_seqlen <= kFwShortPrompt) {
    FsOrder o;
    o.n_heads = c.n_heads * c.group;
    o.units = c.units * c.group;
    o.kv_div = c.group;
    o.grp = s.fs_grp;
    o.n_groups = s.fs_groups;
    o.n_items = s.fs_items;
    o.item_base = s.item_base;
    const int n_items = o.n_items;
    if (n_items == 0) return cudaSuccess;
    const int smem = kTileBytes + kFsKvSlots * kFwKvSlotBytes + 1024;
    static unsigned long long attr_flags = 0;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(fwd_tc_short_kernel), smem, &attr_flags);
    if (e != cudaSuccess) return e;
    const int blocks = n_items < 2 * sm_count() ? n_items : 2 * sm_count();
    fwd_tc_short_kernel<<<blocks, kFsThreads, smem, stream>>>(map_q, map_k, map_v, s, o, make_scale2(c.scale),
                                                              static_cast<__nv_bfloat16*>(out), c.status);
    return cudaGetLastError();
  }
  return launch_fwd_g<2>(map_q, map_k, map_v, c, s, max_seqlen, out, stream);
}

// Units per group of the persistent forward kernel's item order (K and V of a group: at most ~48 MB, well
// inside the L2); 0: this prompt length does not use that kernel.
int fwd_group_units(int units, int max_seqlen) {
  if (max_seqlen > kFwShortPrompt) return 0;
  const int nb_max = (max_seqlen + kTile - 1) / kTile;
  const int64_t unit_bytes = (int64_t)nb_max * kTile * kD * 2 * 2;
  return (int)std::max<int64_t>(1, std::min<int64_t>(units, (48ll << 20) / unit_bytes));
}

bool prefill_tc_supported(int dtype, int head_dim) { return dtype == H2O_BF16 && head_dim == kD && encode_fn() != nullptr; }

cudaError_t launch_colsum_tc(const CacheView& c, const PrefillScratch& s, int max_seqlen, const void* q, const void* k,
                             cudaStream_t stream) {
  CUtensorMap map_q, map_k;
  if (!make_whole_tile_map(&map_q, q, s.total_tokens, c.n_heads * c.group, kTile) ||
      !make_whole_tile_map(&map_k, k, s.total_tokens, c.n_heads, kTile))
    return cudaErrorInvalidValue;
  const int smem = kTileBytes * (1 + kCsQStages) + 1024;
  static unsigned long long attr_flags = 0;
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(colsum_tc_kernel), smem, &attr_flags);
    if (e != cudaSuccess) return e;
  }
  const int nb = (max_seqlen + kTile - 1) / kTile;
  const int max_pairs = (nb + 1) / 2, n_items = max_pairs * c.units;
  if (n_items == 0) return cudaSuccess;
  // Short prompts (few tiles per item): persistent blocks, two per SM (256 TMEM columns, 97 KB of shared
  // memory each), so that an item's fixed cost (first loads, pipeline fill) overlaps the previous item's
  // last tiles: config 3 (five tiles per item) 273 -> 250 us.  Long items run one per block and leave the
  // balancing to the hardware scheduler (config 2, 17 tiles per item: 212 us against 216 us persistent).
  const bool persistent = c.group * (nb + 1) <= kCsPersistentTiles && n_items > 2 * sm_count();
  const int blocks = persistent ? 2 * sm_count() : n_items;
  colsum_tc_kernel<<<blocks, kCsThreads, smem, stream>>>(map_q, map_k, s, c.n_heads, c.group, max_pairs, n_items,
                                                         make_scale2(c.scale), c.status);
  return cudaGetLastError();
}

}  // namespace h2o
