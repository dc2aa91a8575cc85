// Decode step and slot gather for caches whose K/V slots are stored 4-bit group-quantised
// (dtype H2O_BF16_KV4: q / k / v / out are bf16, head_dim 128).
//
// The paper states that the eviction policy combines with 4-bit quantisation (Q3 of its question section,
// appendix on throughput with quantisation) without giving a quantiser; the one used here is this library's
// own.  A stored row of 128 channels is 80 bytes:
//   bytes  0..63   codes, channel c in byte c / 2 (even channel: low nibble); group g = channels 32 g .. 32 g + 31
//                  = bytes 16 g .. 16 g + 15
//   bytes 64..79   per group g: scale (bf16), zero (bf16)
// and, in fp32 with round-to-nearest-even throughout,
//   zero  = min of the group (an input value)          scale = bf16((max - zero) / 15), 1 for a constant group
//   code  = clamp(rint((x - zero) / scale), 0, 15)      x_hat = zero + code * scale
// A row is quantised when it enters the cache: the kept prompt rows at the gather, a new token's row after
// its own step, in which it still takes part at full precision.
//
// The decode step is the same fused step as decode.cu (scores over the occupied slots, softmax, P V,
// fp64 score accumulation, victim search, in-place write), with the dequantisation folded into the
// arithmetic: per group  q . x_hat = zero * sum(q) + scale * sum(q_i code_i)  and
// sum_rows p * x_hat_i = sum_rows (p * scale) * code_i + sum_rows p * zero.  Both contractions over codes run
// as mma.sync m16n8k16 on the codes as exact bf16 values (the unpacking, one shift and one logic operation
// per pair of codes, is what bounds the kernel: the logic pipe, not HBM): the scores with the query as the
// column operand, one column per group; the values with the codes transposed as the row operand and
// p * scale, split into a bf16 head and remainder per group, as the column operand.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <climits>
#include <cmath>
#include <cstdint>

#include "h2o.h"
#include "h2o_internal.cuh"
#include "sm100_ptx.cuh"
#include "step_common.cuh"

namespace cg = cooperative_groups;

namespace h2o {
namespace {

using namespace ptx;

constexpr int kMaxSplit = 8;
using namespace step;

constexpr int kD = 128;
constexpr int kRowBytes = 80;
constexpr int kMaxWarps = 16;             // consumer warps: 16 when a block has its SM to itself, 8 for two blocks per
                                          // SM, 4 for launches of many units (more blocks per SM hide one another's
                                          // serial start and end); one more warp streams the tiles
constexpr int kTileRows = 64;             // rows per tile: eight per consumer warp
constexpr int kTileBytes = kTileRows * kRowBytes;  // 5120
constexpr int kMaxStages = 8;             // ring depth: 2, 4 or 8 tiles (K and V) in flight
// (a & b) | c in one logic instruction
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// The eight codes of a 32-bit word as four pairs of exact bf16 values, r[k] = (code k, code k + 4): a nibble in
// the low mantissa bits of 128.0 reads as 128 + code; the subtraction is exact.
__device__ __forceinline__ void codes_bf16x2(uint32_t w, uint32_t (&r)[4]) {
  const __nv_bfloat162 c128 = __floats2bfloat162_rn(128.f, 128.f);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    uint32_t x = and_or(w >> (4 * k), 0x000F000Fu, 0x43004300u);
    __nv_bfloat162 v = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&x), c128);
    r[k] = *reinterpret_cast<uint32_t*>(&v);
  }
}
// D (16 x 8, fp32) += A (16 x 16, bf16, row) * B (16 x 8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

// Quantise one group of 32 channels (bf16 inputs); codes: 16 bytes, meta = scale | zero << 16 (bf16 bits).
__device__ __forceinline__ void quantise_group(const __nv_bfloat16* src, uint4& codes, uint32_t& meta) {
  float x[32];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 raw = *reinterpret_cast<const uint4*>(src + 8 * i);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      x[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
      x[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
  float mn = x[0], mx = x[0];
#pragma unroll
  for (int i = 1; i < 32; ++i) {
    mn = fminf(mn, x[i]);
    mx = fmaxf(mx, x[i]);
  }
  float scale = __bfloat162float(__float2bfloat16_rn(__fdiv_rn(__fsub_rn(mx, mn), 15.0f)));
  if (!(scale > 0.f)) scale = 1.0f;
  uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    float t = rintf(__fdiv_rn(__fsub_rn(x[i], mn), scale));
    t = fminf(fmaxf(t, 0.f), 15.f);
    w[i >> 3] |= (uint32_t)t << (4 * (i & 7));
  }
  codes = make_uint4(w[0], w[1], w[2], w[3]);
  meta = (__float_as_uint(scale) >> 16) | (__float_as_uint(mn) & 0xffff0000u);
}

#ifdef H2O_PHASE_TIMERS
__device__ long long g_kvt[512 * 2 * 16];
#define KV_STAMP(i)                                                                              \
  do {                                                                                           \
    if (lane == 0 && (warp == 0 || warp == 4) && blockIdx.x < 512 && (i) < 16) {                \
      long long ts_;                                                                             \
      asm volatile("mov.u64 %0, %%clock64;" : "=l"(ts_));                                       \
      g_kvt[(blockIdx.x * 2 + (warp >> 2)) * 16 + (i)] = ts_;                                     \
    }                                                                                            \
  } while (0)
#else
#define KV_STAMP(i) do { } while (0)
#endif

struct Shared {
  uint64_t full[kMaxStages], empty[kMaxStages], aux;
  uint64_t nr;  // the producer warp has quantised the new token's row
  float red[kMaxWarps][kD];  // per-warp partial outputs (unnormalised, relative to the warp's maximum)
  float gm[kMaxWarps], gl[kMaxWarps];
  Cand wbest[kMaxWarps];
  __align__(16) unsigned char newrow[2][kRowBytes];  // the new token's K and V row, quantised
  // the query as the B operand of the score products, per lane 16 words (rows padded to 20 words: 16-byte
  // reads of eight consecutive lanes then fall into different banks)
  __align__(16) uint32_t qb[32][20];
  // Cluster exchange (a unit split over the blocks of a cluster, CLUSTER instances): every block pushes its values
  // into its peers' shared memory with remote stores, then one cluster barrier makes them visible.
  float x_m[kMaxSplit], x_l[kMaxSplit];  // block statistics of every rank (written by that rank)
  float x_out[kMaxSplit][kD];            // rank 0 only: every rank's partial output, relative to its own maximum
  Cand x_cand[kMaxSplit];                // rank 0 only: every rank's eviction candidate
};

// MINB: blocks per SM the register allocation leaves room for (the kernel wants ~96 registers a thread).
// EARLY: the instances for launches of at most two waves of blocks, where the start of a block is exposed: they
// take the host's hints (cache untouched by the previous launch of the stream: tiles requested before the grid
// dependency is awaited; every unit full: no counter read before the first request) and fetch the new value row
// at the start.  In launches of many waves the same code was slower
// (3584 units of 104 slots: 46.4 -> 48.4 us), so those instances leave it out.
// CLUSTER: the instance that splits a unit over the blocks of a cluster (few long units): block `rank` owns slots
// rank * chunk .. of the unit; statistics and partial outputs are exchanged after the stream, candidates after the
// final probabilities, as in the step kernel of the bf16 slots.
template <int MINB, int kWarps, bool EARLY, bool CLUSTER>
__global__ void __launch_bounds__(kWarps * 32 + 32, MINB)
decode_kv4_kernel(CacheView c, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_new,
                  const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ out,
                  int32_t* __restrict__ evicted_pos, int split_arg, int chunk, int stage_shift, int launch_flags) {
  const int split = CLUSTER ? split_arg : 1;
  constexpr int kThreads = kWarps * 32;
  const int stages = 1 << stage_shift;  // ring depth: a power of two
  extern __shared__ __align__(128) unsigned char dyn[];
  __shared__ Shared sh;
  // dynamic layout: ring[stages][K tile | V tile] | acc_s[chunk] f64 | pos_s[chunk] i32 | p[chunk] f32
  unsigned char* ring = dyn;
  double* acc_s = reinterpret_cast<double*>(dyn + (size_t)stages * 2 * kTileBytes);
  int32_t* pos_s = reinterpret_cast<int32_t*>(acc_s + chunk);
  float* p = reinterpret_cast<float*>(pos_s + chunk);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = split > 1 ? (int)cluster.block_rank() : 0;
  // Early arrival on the cluster barrier; the matching wait comes right before the first remote store.
  if (split > 1) cluster.barrier_arrive();
  const int su = blockIdx.x / split;
  const int lo = rank * chunk;  // first slot of this block
  const UnitMeta mt = c.meta[su];
  // Programmatic dependent launch, as in the step kernel of the bf16 slots: the inputs may come from the previous
  // kernel of the stream and are read after griddepcontrol.wait; the cache is written by this library alone, and
  // when the host knows that its previous launch on this stream wrote another cache (`cache_is_quiescent`) the
  // tiles are requested before the wait.  When the host expects every unit to be full (`all_full`) the block
  // streams its whole budget without reading the counter first; the expectation only decides what is fetched.
  bool cache_is_quiescent = false, all_full = false;
  if constexpr (EARLY) {
    cache_is_quiescent = (launch_flags & 1) != 0;
    all_full = (launch_flags & 2) != 0;
  }
  if (!cache_is_quiescent) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  KV_STAMP(13);
  const int u = mt.unit, r = mt.rwin, B = mt.kbud + mt.rwin;
  int cnt_u, cnt, nstr;  // entries of the unit, of this block, rows to stream
  if constexpr (EARLY) {
    cnt_u = all_full ? 0 : c.count[su];
    nstr = all_full ? max(0, min(B - lo, chunk)) : max(0, min(cnt_u - lo, chunk));
  } else {
    cnt_u = c.count[su];
    nstr = CLUSTER ? max(0, min(cnt_u - lo, chunk)) : cnt_u;
  }
  const int t = c.tpos[su];
  // (checked build: the unit and the rows this block streams must lie inside the cache)
  if (!H2O_IN_RANGE(mt.unit, c.units, c.status) || !H2O_IN_RANGE(nstr, min(B, chunk) + 1, c.status) ||
      !H2O_IN_RANGE(mt.slot_off + lo + (nstr > 0 ? nstr - 1 : 0), c.total_slots, c.status))
    nstr = 0;
  const int ntile = (nstr + kTileRows - 1) / kTileRows;
  unsigned char* Kb = static_cast<unsigned char*>(c.K) + (mt.slot_off + lo) * kRowBytes;
  unsigned char* Vb = static_cast<unsigned char*>(c.V) + (mt.slot_off + lo) * kRowBytes;
  double* acc_g = c.acc + mt.slot_off + lo;
  int32_t* pos_g = c.pos + mt.slot_off + lo;
  const __nv_bfloat16* qu = q + (int64_t)u * kD;
  const __nv_bfloat16* ku = k_new + (int64_t)u * kD;
  const __nv_bfloat16* vu = v_new + (int64_t)u * kD;
  bool timed_out = false;
  // the consumer lanes' query and new-key words (the sixteen channels 16 (lane % 8) .. for the self score, the
  // group 32 c4 .. for the operands) and warp 0's words of the new value: requested as early as the launch
  // order allows, so that their latency overlaps the block's start
  uint4 in_q[2], in_k[2], in_g[4];
  uint2 in_v = make_uint2(0u, 0u);
  auto load_inputs = [&]() {
    if (warp < kWarps) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        in_q[i] = *reinterpret_cast<const uint4*>(qu + 16 * (lane & 7) + 8 * i);
        in_k[i] = *reinterpret_cast<const uint4*>(ku + 16 * (lane & 7) + 8 * i);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) in_g[i] = *reinterpret_cast<const uint4*>(qu + 32 * (lane & 3) + 8 * i);
      if (EARLY && warp == 0) in_v = *reinterpret_cast<const uint2*>(vu + 4 * lane);
    }
  };
  if (!cache_is_quiescent) load_inputs();

  auto issue_stage = [&](int j) {  // producer lane only
    const int s = j & (stages - 1);
    const int rows = min(kTileRows, nstr - j * kTileRows);
    const uint32_t bytes = (uint32_t)rows * kRowBytes;
    unsigned char* dst = ring + (size_t)s * 2 * kTileBytes;
    mbar_expect_tx(&sh.full[s], 2 * bytes);
    bulk_load(dst, Kb + (size_t)j * kTileBytes, bytes, &sh.full[s]);
    bulk_load(dst + kTileBytes, Vb + (size_t)j * kTileBytes, bytes, &sh.full[s]);
  };
  if (tid == kThreads) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], 4);  // a tile is consumed by four warps
    }
    mbar_init(&sh.aux, 1);
    mbar_init(&sh.nr, 1);
    fence_barrier_init();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int j = 0; j < min(stages, ntile); ++j) issue_stage(j);
    if (nstr > 0) {
      const int npad = (nstr + 3) & ~3;  // stays inside the unit's padded slot range
      mbar_expect_tx(&sh.aux, (uint32_t)npad * 12u);
      bulk_load(acc_s, acc_g, (uint32_t)npad * 8u, &sh.aux);
      bulk_load(pos_s, pos_g, (uint32_t)npad * 4u, &sh.aux);
    }
  }
  if constexpr (EARLY) {
    if (all_full) cnt_u = c.count[su];
  }
  if constexpr (EARLY) cnt = max(0, min(min(cnt_u - lo, chunk), nstr));  // (never more than was streamed)
  else cnt = nstr;
  __syncthreads();
  if constexpr (EARLY) {
    if (cache_is_quiescent) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      load_inputs();
    }
  }

  if (warp == kWarps) {
    // ---- producer warp: one lane streams the tiles; lanes 0..7 quantise the new token's row meanwhile ----
    if (lane < 8) {
      uint4 codes;
      uint32_t meta;
      quantise_group((lane < 4 ? ku : vu) + 32 * (lane & 3), codes, meta);
      unsigned char* row = sh.newrow[lane >> 2];
      *reinterpret_cast<uint4*>(row + 16 * (lane & 3)) = codes;
      *reinterpret_cast<uint32_t*>(row + 64 + 4 * (lane & 3)) = meta;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.nr);
    if (lane == 0) {
      for (int j = stages; j < ntile; ++j) {
        if (!bar_wait(&sh.empty[j & (stages - 1)], (uint32_t)((j >> stage_shift) - 1) & 1u)) timed_out = true;
        issue_stage(j);
      }
      if (timed_out) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
    }
    __syncwarp();
    if (split > 1) {  // the producer warp only keeps the cluster barriers balanced (both exchanges follow the stream)
      cluster.barrier_wait();
      cluster.sync();
      cluster.sync();
    }
  } else {
    // ---- consumer warps --------------------------------------------------------------------------
    // A warp takes 16 rows of a tile (with eight warps: warps 0..3 the even tiles, warps 4..7 the odd ones).
    // Scores on the tensor cores (mma.sync m16n8k16, bf16 x bf16 -> fp32; codes 0..15 are exact in bf16):
    // A = the codes of 16 rows x 16 channels, B = the query with column n = quantisation group (zero outside
    // the group), so that one accumulator tile holds, per row, the four group sums  sum(q_i code_i);
    // scale and zero are applied once per group.  Lane (g, c4) = (lane / 4, lane % 4) loads the 16 bytes of
    // group c4 of rows g and g + 8; which channel sits at which k index is free as long as B agrees.
    // Values on the tensor cores as well, with the codes as the row operand and the weights as the column operand.
    const int g = lane >> 2, c4 = lane & 3;
    // the new token against itself, at full precision (every warp computes the same value)
    float s_self;
    {
      float part = 0.f;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint4 rq = in_q[i], rk = in_k[i];
        const uint32_t wq[4] = {rq.x, rq.y, rq.z, rq.w}, wk[4] = {rk.x, rk.y, rk.z, rk.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          part = fmaf(__uint_as_float(wq[j] << 16), __uint_as_float(wk[j] << 16), part);
          part = fmaf(__uint_as_float(wq[j] & 0xffff0000u), __uint_as_float(wk[j] & 0xffff0000u), part);
        }
      }
      part += __shfl_xor_sync(0xffffffffu, part, 1);
      part += __shfl_xor_sync(0xffffffffu, part, 2);
      part += __shfl_xor_sync(0xffffffffu, part, 4);
      s_self = rank == 0 ? c.scale * part : -INFINITY;  // (split unit: the first block's entry)
    }
    // the query of group c4: its sum, and (warp 0) its words as B operands.  For the word w of a row
    // (channels 8 w .. 8 w + 7 of the group) the two products use k index pairs (code 0, code 4 | code 1,
    // code 5) and (code 2, code 6 | code 3, code 7), see codes_bf16x2.
    float qsA, qsB;  // query sums of groups 2 c4 and 2 c4 + 1 (used by c4 < 2)
    {
      uint32_t raw[16];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 r4 = in_g[i];
        raw[4 * i] = r4.x;
        raw[4 * i + 1] = r4.y;
        raw[4 * i + 2] = r4.z;
        raw[4 * i + 3] = r4.w;
      }
      float qs = 0.f;
#pragma unroll
      for (int i = 0; i < 16; ++i) qs += __uint_as_float(raw[i] << 16) + __uint_as_float(raw[i] & 0xffff0000u);
      qsA = __shfl_sync(0xffffffffu, qs, (lane & ~3) | ((2 * c4) & 3));
      qsB = __shfl_sync(0xffffffffu, qs, (lane & ~3) | ((2 * c4 + 1) & 3));
      if (warp == 0) {
        const bool mine = g == c4;  // column n = g of B is group g: only the lanes that hold that group's channels
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          uint4 b;
          b.x = mine ? __byte_perm(raw[4 * w], raw[4 * w + 2], 0x5410) : 0u;
          b.y = mine ? __byte_perm(raw[4 * w], raw[4 * w + 2], 0x7632) : 0u;
          b.z = mine ? __byte_perm(raw[4 * w + 1], raw[4 * w + 3], 0x5410) : 0u;
          b.w = mine ? __byte_perm(raw[4 * w + 1], raw[4 * w + 3], 0x7632) : 0u;
          *reinterpret_cast<uint4*>(&sh.qb[lane][4 * w]) = b;
        }
      }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
    float o[32];  // o[4 j + i] = accumulator i of the value product j (see below)
#pragma unroll
    for (int i = 0; i < 32; ++i) o[i] = 0.f;
    float zacc = 0.f;  // sum of p * zero of this lane's rows and group, minus the code offset's share
    float mg = -INFINITY, lg = 0.f;
    const int cb = (warp & 3) * 16;  // the warp's rows of a tile
    KV_STAMP(0);
    for (int j = warp >> 2; j < ntile; j += kWarps / 4) {
      const int s = j & (stages - 1);
      if (!bar_wait(&sh.full[s], (uint32_t)(j >> stage_shift) & 1u)) timed_out = true;
      KV_STAMP(1 + 3 * (j / (kWarps / 4)));
      const unsigned char* kt = ring + (size_t)s * 2 * kTileBytes;
      const unsigned char* vt = kt + kTileBytes;
      const int rows = min(kTileRows, cnt - j * kTileRows);
      // ---- scores of rows cb + g and cb + g + 8 ----
      const int rowA = cb + g, rowB = rowA + 8;
      float sA, sB;
      {
        const uint4 ka = *reinterpret_cast<const uint4*>(kt + rowA * kRowBytes + 16 * c4);
        const uint4 kb = *reinterpret_cast<const uint4*>(kt + rowB * kRowBytes + 16 * c4);
        const uint32_t wa[4] = {ka.x, ka.y, ka.z, ka.w}, wb[4] = {kb.x, kb.y, kb.z, kb.w};
        float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};  // two chains
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          uint32_t ra[4], rb[4];
          codes_bf16x2(wa[w], ra);
          codes_bf16x2(wb[w], rb);
          const uint4 b = *reinterpret_cast<const uint4*>(&sh.qb[lane][4 * w]);
          mma_bf16_16816(d0, ra[0], rb[0], ra[1], rb[1], b.x, b.y);
          mma_bf16_16816(d1, ra[2], rb[2], ra[3], rb[3], b.z, b.w);
        }
        // lanes c4 < 2 hold the sums of groups 2 c4 and 2 c4 + 1 (columns 4..7 of the tile are zero)
        const uint2 ma = *reinterpret_cast<const uint2*>(kt + rowA * kRowBytes + 64 + 8 * (c4 & 1));
        const uint2 mb = *reinterpret_cast<const uint2*>(kt + rowB * kRowBytes + 64 + 8 * (c4 & 1));
        // q . x_hat = zero sum(q) + scale sum(q_i code_i), per group
        float pa = fmaf(bf16_bits_to_float(ma.x & 0xffffu), d0[0] + d1[0], bf16_bits_to_float(ma.x >> 16) * qsA);
        pa += fmaf(bf16_bits_to_float(ma.y & 0xffffu), d0[1] + d1[1], bf16_bits_to_float(ma.y >> 16) * qsB);
        float pb = fmaf(bf16_bits_to_float(mb.x & 0xffffu), d0[2] + d1[2], bf16_bits_to_float(mb.x >> 16) * qsA);
        pb += fmaf(bf16_bits_to_float(mb.y & 0xffffu), d0[3] + d1[3], bf16_bits_to_float(mb.y >> 16) * qsB);
        if (c4 >= 2) {
          pa = 0.f;
          pb = 0.f;
        }
        pa += __shfl_xor_sync(0xffffffffu, pa, 1);
        pb += __shfl_xor_sync(0xffffffffu, pb, 1);
        pa += __shfl_xor_sync(0xffffffffu, pa, 2);
        pb += __shfl_xor_sync(0xffffffffu, pb, 2);
        // (rows past the end hold stale bytes: whatever they gave is dropped here)
        sA = rowA < rows ? c.scale * pa : -INFINITY;
        sB = rowB < rows ? c.scale * pb : -INFINITY;
        if (c4 == 0) {  // raw scores, finalised after the stream
          if (rowA < rows) p[j * kTileRows + rowA] = sA;
          if (rowB < rows) p[j * kTileRows + rowB] = sB;
        }
      }
      KV_STAMP(2 + 3 * (j / (kWarps / 4)));
      // one softmax state per warp: maximum over its sixteen rows of this tile
      float mnew = fmaxf(mg, fmaxf(sA, sB));
      mnew = fmaxf(mnew, __shfl_xor_sync(0xffffffffu, mnew, 4));
      mnew = fmaxf(mnew, __shfl_xor_sync(0xffffffffu, mnew, 8));
      mnew = fmaxf(mnew, __shfl_xor_sync(0xffffffffu, mnew, 16));
      if (mnew > -INFINITY) {  // warp-uniform
        const float f = expf(mg - mnew);  // expf(-inf) = 0 for the warp's first rows
        const float eA = expf(sA - mnew), eB = expf(sB - mnew);  // 0 for rows past the end
        float esum = eA + eB;  // over the warp's rows (the four lanes of a group hold the same values)
        esum += __shfl_xor_sync(0xffffffffu, esum, 4);
        esum += __shfl_xor_sync(0xffffffffu, esum, 8);
        esum += __shfl_xor_sync(0xffffffffu, esum, 16);
        lg = fmaf(lg, f, esum);
        zacc *= f;
        if (f != 1.0f) {  // (warp-uniform) the reference maximum moved
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] *= f;
        }
        // ---- values on the tensor cores: D[channel][column] += codes^T[channel][row] * W[row][column] ----
        // k = the warp's sixteen rows; m = sixteen channels per product j: channel 8 g + j (word g of the
        // row, nibble j) and 64 + 8 g + j (word g + 8); n = (group, part): column grp + 4 part holds the
        // weight p * scale of (row, grp) split into a bf16 head (part 0) and its bf16 remainder (part 1).
        // Codes enter as 128 + code (exact in bf16); the offset's share 128 * (sum of the weights as given)
        // leaves through zacc together with the zeros.  Lane (g, c4) holds rows 2 c4, 2 c4 + 1, 2 c4 + 8,
        // 2 c4 + 9 for both operands; its column of W is n = g.
        const int grp = g & 3;
        const bool head = g < 4;
        float part[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int rr = 2 * c4 + (x & 1) + 8 * (x >> 1);
          const float e = __shfl_sync(0xffffffffu, x < 2 ? eA : eB, 4 * (2 * c4 + (x & 1)));
          uint32_t vmeta = *reinterpret_cast<const uint32_t*>(vt + (cb + rr) * kRowBytes + 64 + 4 * grp);
          if (cb + rr >= rows) vmeta = 0u;  // stale bytes past the end of the last tile
          const float w = e * bf16_bits_to_float(vmeta & 0xffffu);
          const float wh = __uint_as_float(__float_as_uint(w) & 0xffff0000u);
          part[x] = head ? wh : w - wh;
          if (head) zacc = fmaf(e, bf16_bits_to_float(vmeta >> 16), zacc);
        }
        uint32_t b0, b1;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(b0) : "f"(part[1]), "f"(part[0]));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(b1) : "f"(part[3]), "f"(part[2]));
        // the offset's share, from the weights as rounded
        zacc -= 128.f * ((__uint_as_float(b0 << 16) + __uint_as_float(b0 & 0xffff0000u)) +
                         (__uint_as_float(b1 << 16) + __uint_as_float(b1 & 0xffff0000u)));
        uint32_t a[4][8];  // [operand register][product j]
#pragma unroll
        for (int hp = 0; hp < 4; ++hp) {  // operand register hp: rows (2 c4, +1) or (2 c4 + 8, +9), word g or g + 8
          const int r0 = cb + 2 * c4 + 8 * (hp >> 1);
          const uint32_t wa = *reinterpret_cast<const uint32_t*>(vt + r0 * kRowBytes + 4 * g + 32 * (hp & 1));
          const uint32_t wb = *reinterpret_cast<const uint32_t*>(vt + (r0 + 1) * kRowBytes + 4 * g + 32 * (hp & 1));
          const uint32_t y0 = __byte_perm(wa, wb, 0x5410), y1 = __byte_perm(wa, wb, 0x7632);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            a[hp][i] = and_or(y0 >> (4 * i), 0x000F000Fu, 0x43004300u);
            a[hp][4 + i] = and_or(y1 >> (4 * i), 0x000F000Fu, 0x43004300u);
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          asm volatile(
              "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
              : "+f"(o[4 * j]), "+f"(o[4 * j + 1]), "+f"(o[4 * j + 2]), "+f"(o[4 * j + 3])
              : "r"(a[0][j]), "r"(a[1][j]), "r"(a[2][j]), "r"(a[3][j]), "r"(b0), "r"(b1));
        }
        mg = mnew;
      }
      __syncwarp();
      KV_STAMP(3 + 3 * (j / (kWarps / 4)));
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&sh.empty[s])) : "memory");
    }
    KV_STAMP(14);
    // zeros and offset: per group, over the warp's rows (the four lanes of a row group) and over head and remainder
    zacc += __shfl_xor_sync(0xffffffffu, zacc, 1);
    zacc += __shfl_xor_sync(0xffffffffu, zacc, 2);
    zacc += __shfl_xor_sync(0xffffffffu, zacc, 16);
    // this lane's column pair is n = 2 c4, 2 c4 + 1: groups 0, 1 (c4 even: channels 8 g + j, accumulators 0 / 1)
    // or 2, 3 (c4 odd: channels 64 + 8 g + j, accumulators 2 / 3); the one that is the channel's own group counts
    const int own = 2 * (c4 & 1) + (g >> 2);
    const float zg = __shfl_sync(0xffffffffu, zacc, 4 * own);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float lo2 = (g >> 2) ? o[4 * j + 1] : o[4 * j], hi2 = (g >> 2) ? o[4 * j + 3] : o[4 * j + 2];
      float v = (c4 & 1) ? hi2 : lo2;
      v += __shfl_xor_sync(0xffffffffu, v, 2);  // head (c4 < 2) + remainder (c4 >= 2)
      if (c4 < 2) sh.red[warp][64 * c4 + 8 * g + j] = v + zg;
    }
    if (lane == 0) {
      sh.gm[warp] = mg;
      sh.gl[warp] = lg;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");

    // ---- block statistics, computed by every warp alike -------------------------------------------
    const float m_i = lane < kWarps ? sh.gm[lane] : -INFINITY;
    float m = m_i;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    m = fmaxf(m, s_self);
    const float w_i = (lane < kWarps && m_i > -INFINITY) ? expf(m_i - m) : 0.f;
    float l = lane < kWarps ? sh.gl[lane] * w_i : 0.f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    float w_self = s_self > -INFINITY ? expf(s_self - m) : 0.f;
    l += w_self;
    float res[4] = {0.f, 0.f, 0.f, 0.f};
    if (warp == 0) {  // the block's output, relative to its maximum: this lane's four channels
      const uint2 raw = EARLY ? in_v : *reinterpret_cast<const uint2*>(vu + 4 * lane);  // the new token's value
      res[0] = w_self * __uint_as_float(raw.x << 16);
      res[1] = w_self * __uint_as_float(raw.x & 0xffff0000u);
      res[2] = w_self * __uint_as_float(raw.y << 16);
      res[3] = w_self * __uint_as_float(raw.y & 0xffff0000u);
#pragma unroll
      for (int g2 = 0; g2 < kWarps; ++g2) {
        const float w = __shfl_sync(0xffffffffu, w_i, g2);
#pragma unroll
        for (int i = 0; i < 4; ++i) res[i] = fmaf(sh.red[g2][4 * lane + i], w, res[i]);
      }
    }
    if (split > 1) {
      const float mc = m, lc = l;
      cluster.barrier_wait();  // every peer is running: its shared memory may be written
      if (tid < split) {       // my statistics into every block of the cluster (my own included)
        *cluster.map_shared_rank(&sh.x_m[rank], tid) = mc;
        *cluster.map_shared_rank(&sh.x_l[rank], tid) = lc;
      }
      if (warp == 0) *reinterpret_cast<float4*>(cluster.map_shared_rank(&sh.x_out[rank][4 * lane], 0)) = make_float4(res[0], res[1], res[2], res[3]);
      cluster.sync();
      const float mr = lane < split ? sh.x_m[lane] : -INFINITY;
      const float lr = lane < split ? sh.x_l[lane] : 0.f;
      m = mr;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
      l = mr > -INFINITY ? lr * expf(mr - m) : 0.f;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
      w_self = s_self > -INFINITY ? expf(s_self - m) : 0.f;
      if (rank == 0 && warp == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) res[i] = 0.f;
        for (int rk = 0; rk < split; ++rk) {
          const float mrk = sh.x_m[rk];
          if (mrk > -INFINITY) {
            const float w = expf(mrk - m);
            const float4 xo = *reinterpret_cast<const float4*>(&sh.x_out[rk][4 * lane]);
            res[0] = fmaf(xo.x, w, res[0]);
            res[1] = fmaf(xo.y, w, res[1]);
            res[2] = fmaf(xo.z, w, res[2]);
            res[3] = fmaf(xo.w, w, res[3]);
          }
        }
      }
    }
    const float inv_l = 1.0f / l;
    if (warp == 0 && rank == 0) {
      uint2 pk;
      pk.x = Vec16<__nv_bfloat16>::pack2(res[0] * inv_l, res[1] * inv_l);
      pk.y = Vec16<__nv_bfloat16>::pack2(res[2] * inv_l, res[3] * inv_l);
      *reinterpret_cast<uint2*>(out + (int64_t)u * kD + 4 * lane) = pk;
    }

    // ---- final probabilities, accumulation (Algorithm 2: accumulated score += probability), victim search ----
    if (nstr > 0 && !bar_wait(&sh.aux, 0)) timed_out = true;
    const bool full = cnt_u >= B;
    const float p_self = w_self * inv_l;
    Cand best = cand_none();
    for (int x = tid; x < cnt; x += kThreads) {
      const float px = expf(p[x] - m) * inv_l;
      const double a = acc_s[x] + (double)px;
      if (H2O_IN_RANGE(mt.slot_off + lo + x, c.total_slots, c.status)) acc_g[x] = a;
      const int ps = pos_s[x];
      if (full && ps <= t - r) {
        const double score = c.score_mode == 1 ? a / (double)(t - ps + 1) : a;
        const Cand cx{(unsigned long long)__double_as_longlong(score), ps, lo + x};
        if (cand_before(cx, best)) best = cx;
      }
    }
    if (rank == 0 && tid == 0 && full && r == 0) {  // without a recent window the new token competes too
      const Cand cs{(unsigned long long)__double_as_longlong((double)p_self), t, -2};
      if (cand_before(cs, best)) best = cs;
    }
    best = warp_argmin(best);
    if (lane == 0) sh.wbest[warp] = best;
    if (timed_out) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
    KV_STAMP(15);
    Cand b = cand_none();
    if (warp == 0) b = warp_argmin(lane < kWarps ? sh.wbest[lane] : cand_none());
    if (split > 1) {
      if (warp == 0 && lane == 0) *cluster.map_shared_rank(&sh.x_cand[rank], 0) = b;
      cluster.sync();  // the last cluster barrier: afterwards rank 0 works on its own memory only
      if (warp == 0 && rank == 0) b = warp_argmin(lane < split ? sh.x_cand[lane] : cand_none());
    }
    if (warp == 0 && rank == 0) {
      int slot, ev;
      if (!full) {
        slot = cnt_u;
        ev = -1;
      } else if (b.slot == -2) {
        slot = -1;
        ev = t;
      } else if (b.slot >= 0) {
        slot = b.slot;
        ev = b.pos;
      } else {  // a full cache always has a candidate; record instead of corrupting
        slot = -1;
        ev = -1;
        if (lane == 0) atomicCAS(c.status, 0, H2O_ERR_STATE);
      }
      if (slot >= 0 && (!H2O_IN_RANGE(slot, B, c.status) || !H2O_IN_RANGE(mt.slot_off + slot, c.total_slots, c.status)))
        slot = -1;  // (checked build) never write outside the unit's slots
      if (lane == 0) {
        if (!full) c.count[su] = cnt_u + 1;
        if (slot >= 0) {
          c.acc[mt.slot_off + slot] = (double)p_self;
          c.pos[mt.slot_off + slot] = t;
        }
        if (evicted_pos) evicted_pos[u] = ev;
        c.tpos[su] = t + 1;
      }
      const bool nr_ok = bar_wait(&sh.nr, 0);  // (long complete: the row was quantised during the stream)
      if (!nr_ok && lane == 0) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
      if (nr_ok && slot >= 0 && lane < 10) {  // the quantised new row goes straight into the freed slot
        const int which = lane / 5, part = lane % 5;  // K: five 16-byte pieces, V: five
        unsigned char* dst = static_cast<unsigned char*>(which == 0 ? c.K : c.V) + (size_t)(mt.slot_off + slot) * kRowBytes + 16 * part;
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(sh.newrow[which] + 16 * part);
      }
    }
  }
}

// Gather of the kept prompt rows into 4-bit slots: one thread per (slot, K or V, group).
__global__ void __launch_bounds__(256)
gather_kv4_kernel(CacheView c, PrefillScratch s, const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v) {
  const int su = blockIdx.x;
  const UnitMeta mt = c.meta[su];
  const int u = mt.unit;
  const int seq = u / c.n_heads, h = u % c.n_heads;
  const int lo = s.cu[seq];
  const int m = c.count[su];
  const int64_t stride = (int64_t)c.n_heads * kD;
  const int64_t base = ((int64_t)lo * c.n_heads + h) * kD;
  unsigned char* Kb = static_cast<unsigned char*>(c.K) + mt.slot_off * kRowBytes;
  unsigned char* Vb = static_cast<unsigned char*>(c.V) + mt.slot_off * kRowBytes;
  for (int x = threadIdx.x; x < m * 8; x += blockDim.x) {
    const int slot = x >> 3, part = x & 7, grp = part & 3;
    if (!H2O_IN_RANGE(mt.slot_off + slot, c.total_slots, c.status)) continue;
    const int j = c.pos[mt.slot_off + slot];
    if (!H2O_IN_RANGE(j, s.cu[seq + 1] - lo, c.status)) continue;  // a kept position is a prompt row of this sequence
    const __nv_bfloat16* src = (part < 4 ? k : v) + base + (int64_t)j * stride + 32 * grp;
    uint4 codes;
    uint32_t meta;
    quantise_group(src, codes, meta);
    unsigned char* row = (part < 4 ? Kb : Vb) + (size_t)slot * kRowBytes;
    *reinterpret_cast<uint4*>(row + 16 * grp) = codes;
    *reinterpret_cast<uint32_t*>(row + 64 + 4 * grp) = meta;
  }
}

}  // namespace

#ifdef H2O_PHASE_TIMERS
extern "C" int h2o_debug_kv4_timers(long long* host, int n) {
  return (int)cudaMemcpyFromSymbol(host, g_kvt, sizeof(long long) * (size_t)n);
}
#endif

size_t kv4_row_bytes() { return kRowBytes; }

template <int MINB, int NW, bool EARLY, bool CLUSTER = false>
static cudaError_t launch_kv4(const CacheView& c, int split, int chunk, int stage_shift, size_t smem, int launch_flags,
                              const void* q, const void* k_new, const void* v_new, void* out, int32_t* evicted_pos,
                              cudaStream_t stream) {
  static unsigned long long attr_flags = 0;  // one word per instance, one bit per device
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_kv4_kernel<MINB, NW, EARLY, CLUSTER>),
                                        200 * 1024, &attr_flags);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(c.units * (CLUSTER ? split : 1)));
  cfg.blockDim = dim3(NW * 32 + 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute at[3];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = (unsigned)split;
  at[1].val.clusterDim.y = 1;
  at[1].val.clusterDim.z = 1;
  // (clusters of a launch should all be resident at once: see the step kernel of decode.cu)
  at[2].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
  at[2].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicyLoadBalancing;
  cfg.attrs = at;
  cfg.numAttrs = (CLUSTER && split > 1) ? 3 : 1;
  return cudaLaunchKernelEx(&cfg, decode_kv4_kernel<MINB, NW, EARLY, CLUSTER>, c, static_cast<const __nv_bfloat16*>(q),
                            static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
                            static_cast<__nv_bfloat16*>(out), evicted_pos, split, chunk, stage_shift, launch_flags);
}

// split: thread blocks (one cluster) per unit, chunk: slots per block (a multiple of 4; the whole budget when split = 1)
cudaError_t launch_decode_kv4(const CacheView& c, int split, int chunk, bool cache_is_quiescent, bool all_full, const void* q,
                              const void* k_new, const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream) {
  if (split < 1 || split > kMaxSplit || (chunk & 3) != 0) return cudaErrorInvalidValue;
  const int launch_flags = (cache_is_quiescent ? 1 : 0) | (all_full ? 2 : 0);
  const int sms = sm_count();
  const int blocks = c.units * split;
  const size_t fixed = (size_t)chunk * 16 + 16;
  auto smem_for = [&](int shift) { return ((size_t)(2 * kTileBytes) << shift) + fixed; };
  if (smem_for(1) > 200 * 1024) return cudaErrorInvalidValue;
#define KV4_GO(M, W, EARLY, CL, SHIFT) \
  return launch_kv4<M, W, EARLY, CL>(c, split, chunk, SHIFT, smem_for(SHIFT), launch_flags, q, k_new, v_new, out, evicted_pos, stream)
  // Few blocks (at most two per SM): the deepest ring that fits, since nothing else hides the load latency
  // (eight tiles in flight against four: 13.1 -> 11.8 us per launch at 256 units of 410 slots); sixteen consumer
  // warps when a block has the SM to itself.
  if (blocks <= 2 * sms) {
    const bool alone = blocks <= sms;
    int shift = 3;
    while (shift > 1 && (alone ? 1 : 2) * (smem_for(shift) + 14 * 1024) > 220 * 1024) --shift;
    if (split > 1) KV4_GO(2, 8, true, true, shift);
    if (alone) KV4_GO(1, 16, true, false, shift);
    KV4_GO(2, 8, true, false, shift);
  }
  // Many blocks: four consumer warps per block and four blocks per SM (96 registers a thread), whose serial
  // starts and ends hide one another; a shallow ring once the blocks outnumber the resident slots.
  if (split > 1) KV4_GO(4, 4, true, true, 1);
  if (blocks > 8 * sms) KV4_GO(4, 4, false, false, 1);
  if (blocks > 4 * sms || smem_for(2) > 200 * 1024) KV4_GO(4, 4, true, false, 1);
  KV4_GO(4, 4, true, false, 2);
#undef KV4_GO
}

// after the selection kernel has written positions, scores and counts (its own row gather is skipped)
cudaError_t launch_gather_kv4(const CacheView& c, const PrefillScratch& s, const void* k, const void* v, cudaStream_t stream) {
  gather_kv4_kernel<<<c.units, 256, 0, stream>>>(c, s, static_cast<const __nv_bfloat16*>(k),
                                                 static_cast<const __nv_bfloat16*>(v));
  return cudaGetLastError();
}

}  // namespace h2o
