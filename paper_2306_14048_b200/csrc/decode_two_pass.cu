// Fused decode step in two streaming passes, bf16 / head_dim 128, for G query heads per (sequence, K/V head) unit:
// G = 1 is plain multi-head attention (Algorithm 2's loop body, as decode.cu: scores over the occupied slots,
// softmax, weighted values, accumulated score += probability, victim, in-place write), G = 2, 4, 8 is
// grouped-query attention, the streaming form of decode_gqa.cu.  The grouped reading is this library's own (the
// paper evicts per head): every query head has its own softmax over the unit's entries, a key's accumulated score
// grows by the sum of the G probabilities (the accumulation once per query head), one victim per unit.
//
// Against the online-softmax kernel of decode.cu this one reads K completely before V: the softmax is exact when
// the values arrive, so the V pass has no running maximum to follow and no rescaling, and the scores come from the
// tensor cores without a shuffle; the price is the pass in between and the scores of all rows in shared memory.
// It is the faster one for launches of more than two blocks per SM unless the units are small.  A unit can be split over the
// blocks of a cluster (few long units): statistics are exchanged between the passes, partial outputs and victim
// candidates in one exchange after the value pass.
//
// Shape: one thread block per unit (or per share of a split unit), eight or four consumer warps and a producer warp.  The producer streams the unit's K
// rows and then its V rows as 8 KB tiles (32 rows) through one bulk-copy ring, so HBM stays busy across the two
// passes.
//   K pass: the scores of 16 rows x G heads are one mma.sync m16n8k16 chain (rows = M, heads = N, channels = K);
//           a lane loads 16 bytes of a row and uses them as the k-slots of two products, the query operand is
//           laid out to match (which channel sits in which k-slot is free as long as both operands agree).  The
//           16-row blocks of the tiles go round the warps.  Raw scores to shared memory, [row][head]; the warps
//           keep the softmax statistics of their rows alongside (one instance computes them in a sweep afterwards).
//   between the passes: the statistics merged per head (exact maximum and sum, as the accumulation needs the final
//           probabilities), one sweep that turns the scores into probabilities in place.
//   V pass: a lane holds eight channels of a row (two rows per warp and pass) and G x 8 accumulators.
// Tail as in the other step kernels: fp64 accumulation of the summed probabilities, victim by (score, position),
// new row written into the freed slot.  Every wait on an mbarrier is bounded (H2O_ERR_TIMEOUT in the status word).
#include <climits>
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "h2o_internal.cuh"
#include "sm100_ptx.cuh"
#include "step_common.cuh"

namespace cg = cooperative_groups;

namespace h2o {

namespace {

using namespace ptx;
using namespace step;

constexpr int kMaxSplit = 8;

constexpr int kD = 128;
constexpr int kTileRows = 32, kRowBytes = kD * 2, kTileBytes = kTileRows * kRowBytes;  // 8 KB
constexpr int kMaxStages = 8;  // ring depth: 8 tiles, or 4 for the four-warp instance (more blocks per SM)
constexpr int kMaxWarps = 8;
template <int THREADS>
__device__ __forceinline__ void consumer_sync_n() { asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory"); }

struct Shared {
  uint64_t full[kMaxStages], empty[kMaxStages], aux;
  float part_m[kMaxWarps][8], part_l[kMaxWarps][8];  // per warp and head: softmax partials
  float m[8], inv_l[8];
  Cand wbest[kMaxWarps];
  // "Top-K" attention: histogram and state of the radix select over the step's logits
  unsigned int hist[256];
  unsigned long long tk_prefix;
  unsigned int tk_remaining, tk_count, tk_bin;  // tk_bin: entries in the bin the last pass chose
  // Cluster exchange (a unit split over the blocks of a cluster): every block pushes its values into its peers'
  // shared memory with remote stores, then one cluster barrier makes them visible.
  float x_m[kMaxSplit][8], x_l[kMaxSplit][8];  // softmax statistics of every rank and head (written by that rank)
  Cand x_cand[kMaxSplit];                      // rank 0 only: every rank's eviction candidate
  // (the partial outputs pushed to rank 0, [kMaxSplit][G][kD] floats, live in dynamic shared memory and exist
  //  only in launches that split a unit)
};

// D (16 x 8, fp32) += A (16 x 16, bf16, row) * B (16 x 8, bf16, col)
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// NW consumer warps: 8 with an 8-deep ring for launches of at most two blocks per SM, 4 with a 4-deep ring otherwise
// (four blocks per SM hide one another's passes between the two streams and their serial ends).  For few units
// neither four warps per block (256 units of 410 slots: 15.4 us against 12.3) nor eight warps capped at 56
// registers with a 4-deep ring, so that the next launch's blocks are resident beside this launch's (14.4 us), helped.
// CLUSTER: the instances that can split a unit over a cluster (the others compile that code out: its registers
// cost the grouped four-warp instance 4 %).
// TOPK: the instances with "Top-K" attention (multi-head, one block per unit): after the K pass the step keeps its
// c.topk largest logits and drops the rest before the statistics.
template <int G, int NW, int STAGES, int MINB, bool CLUSTER, bool TOPK>
__global__ void __launch_bounds__(NW * 32 + 32, MINB)
decode_two_pass_kernel(CacheView c, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_new,
                       const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ out,
                       int32_t* __restrict__ evicted_pos, int split_arg, int chunk, int launch_flags) {
  const int split = CLUSTER ? split_arg : 1;
  constexpr int kWarps = NW, kThreads = NW * 32, kStages = STAGES, kStageShift = STAGES == 8 ? 3 : 2;
  // KSTATS: the warps keep the softmax statistics of their rows during the K pass (see there).  Not in the
  // instance of many large multi-head units: with one head three quarters of the lanes' work on the statistics
  // is idle, and where several waves of blocks hide the pass between the streams anyway the extra instructions
  // cost more than the shorter pass saves (config 5: 139.7 against 142.2 us); everywhere else it wins (3584 units
  // of 104 slots: 45.6 -> 42.1 us; 512 grouped units, G = 8: 31.9 -> 29.8 us).
  constexpr bool KSTATS = !TOPK && !(G == 1 && NW == 4 && MINB == 4);  // ("Top-K": the statistics follow the selection)
  auto consumer_sync = [] { consumer_sync_n<NW * 32>(); };
  extern __shared__ __align__(128) unsigned char dyn[];
  __shared__ Shared sh;
  // dynamic layout: ring[kStages][tile] (reused for the warps' partial outputs after the stream) |
  //                 acc_s[chunk] f64 | pos_s[chunk] i32 | p[(chunk + 4) * G] f32 ([row][head]; row cnt = the token itself)
  unsigned char* ring = dyn;
  double* acc_s = reinterpret_cast<double*>(dyn + (size_t)kStages * kTileBytes);
  int32_t* pos_s = reinterpret_cast<int32_t*>(acc_s + chunk);
  float* p = reinterpret_cast<float*>(pos_s + chunk);
  float* red = reinterpret_cast<float*>(ring);  // [2 * kWarps][G][kD]
  float* x_out = p + (size_t)(chunk + 4) * G;   // [kMaxSplit][G][kD], only when split > 1

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = split > 1 ? (int)cluster.block_rank() : 0;
  // Early arrival on the cluster barrier; the matching wait comes right before the first remote store, by which
  // time every block of the cluster has long started (its shared memory exists).
  if (split > 1) cluster.barrier_arrive();
  const int su = blockIdx.x / split;  // launch position of the unit; the block owns rows lo .. lo + chunk - 1 of it
  const int lo = rank * chunk;
  const UnitMeta mt = c.meta[su];
  // Programmatic dependent launch, as in the multi-head step kernel: the inputs may come from the previous kernel
  // of the stream and are read after griddepcontrol.wait; the cache is written by this library alone, and when the
  // host knows that its previous launch on this stream wrote another cache (`cache_is_quiescent`) the first tiles
  // are requested before the wait.  When the host expects every unit to be full (`all_full`) the block streams its
  // whole budget without reading the counter first; the expectation only decides what is fetched.
  const bool cache_is_quiescent = (launch_flags & 1) != 0, all_full = (launch_flags & 2) != 0;
  if (!cache_is_quiescent) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  const int u = mt.unit, r = mt.rwin, B = mt.kbud + mt.rwin;
  int cnt_u = all_full ? 0 : c.count[su];  // entries of the unit
  const int t = c.tpos[su];
  int nstr = all_full ? max(0, min(min(B, split * chunk) - lo, chunk)) : max(0, min(cnt_u - lo, chunk));  // rows to stream
  if (!H2O_IN_RANGE(u, c.units, c.status) || !H2O_IN_RANGE(nstr, chunk + 1, c.status) ||
      (nstr > 0 && !H2O_IN_RANGE(mt.slot_off + lo + nstr - 1, c.total_slots, c.status)))
    nstr = 0;
  const int nt = (nstr + kTileRows - 1) / kTileRows;  // tiles per matrix; the stream is K 0..nt-1, then V 0..nt-1
  const __nv_bfloat16* Kb = reinterpret_cast<const __nv_bfloat16*>(c.K) + (mt.slot_off + lo) * kD;
  const __nv_bfloat16* Vb = reinterpret_cast<const __nv_bfloat16*>(c.V) + (mt.slot_off + lo) * kD;
  double* acc_g = c.acc + mt.slot_off + lo;
  int32_t* pos_g = c.pos + mt.slot_off + lo;
  const __nv_bfloat16* qu = q + (int64_t)u * G * kD;  // the group's query heads are consecutive
  const __nv_bfloat16* ku = k_new + (int64_t)u * kD;
  const __nv_bfloat16* vu = v_new + (int64_t)u * kD;
  bool timed_out = false;

  // the query operand of the score products: lane (n, c4) = (lane / 4, lane % 4) holds head n's channels
  // 32 cc + 8 c4 .. + 7 for cc = 0..3 (zeros for n >= G), the same bytes a lane loads of a key row
  const int gl = lane >> 2, c4 = lane & 3;
  uint4 qb[4];
  auto load_query = [&]() {
#pragma unroll
    for (int cc = 0; cc < 4; ++cc)
      qb[cc] = (warp < kWarps && gl < G) ? *reinterpret_cast<const uint4*>(qu + gl * kD + 32 * cc + 8 * c4) : make_uint4(0, 0, 0, 0);
  };
  if (!cache_is_quiescent) load_query();

  auto issue_tile = [&](int T) {  // producer lane only
    const int s = T & (kStages - 1);
    const int j = T < nt ? T : T - nt;
    const int rows = min(kTileRows, nstr - j * kTileRows);
    const uint32_t bytes = (uint32_t)rows * kRowBytes;
    mbar_expect_tx(&sh.full[s], bytes);
    bulk_load(ring + (size_t)s * kTileBytes, (T < nt ? Kb : Vb) + (int64_t)j * kTileRows * kD, bytes, &sh.full[s]);
  };
  if (tid == kThreads) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], kWarps);
    }
    mbar_init(&sh.aux, 1);
    fence_barrier_init();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int T = 0; T < min(kStages, 2 * nt); ++T) issue_tile(T);
    if (nstr > 0) {
      const int npad = (nstr + 3) & ~3;  // stays inside the unit's padded slot range
      mbar_expect_tx(&sh.aux, (uint32_t)npad * 12u);
      bulk_load(acc_s, acc_g, (uint32_t)npad * 8u, &sh.aux);
      bulk_load(pos_s, pos_g, (uint32_t)npad * 4u, &sh.aux);
    }
  }
  if (all_full) cnt_u = c.count[su];
  if (!H2O_IN_RANGE(cnt_u, B + 1, c.status)) cnt_u = 0;  // (checked build) a unit never holds more than its budget
  const int cnt = max(0, min(min(cnt_u - lo, chunk), nstr));  // occupied rows of this block
  __syncthreads();
  if (cache_is_quiescent) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    load_query();
  }

  if (warp == kWarps) {
    // ---- producer warp: one lane keeps the ring full ------------------------------------------------------
    // (Split unit: the warp has nothing to exchange and only keeps the cluster barriers balanced.  It must not
    //  stand in the barrier between the passes while value tiles are still to be requested: the consumers reach
    //  that barrier before they free the slots those tiles need.  So it completes the first barrier at once,
    //  arrives on the second without waiting, streams, and waits afterwards.)
    if (split > 1) {
      cluster.barrier_wait();
      cluster.barrier_arrive();
    }
    if (lane == 0) {
      for (int T = kStages; T < 2 * nt; ++T) {
        if (!bar_wait(&sh.empty[T & (kStages - 1)], (uint32_t)((T >> kStageShift) - 1) & 1u)) timed_out = true;
        issue_tile(T);
      }
      if (timed_out) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
    }
    __syncwarp();
    if (split > 1) {
      cluster.barrier_wait();
      cluster.sync();
    }
    return;
  }

  // ---- consumer warps -------------------------------------------------------------------------------------
  // the new token against itself, per query head (the heads go round the warps), with plain arithmetic
  for (int g = warp; g < G && rank == 0; g += kWarps) {  // (with a split unit: the first block's entry)
    const uint2 rq = *reinterpret_cast<const uint2*>(qu + g * kD + 4 * lane);
    const uint2 rk = *reinterpret_cast<const uint2*>(ku + 4 * lane);
    float part = __uint_as_float(rq.x << 16) * __uint_as_float(rk.x << 16);
    part = fmaf(__uint_as_float(rq.x & 0xffff0000u), __uint_as_float(rk.x & 0xffff0000u), part);
    part = fmaf(__uint_as_float(rq.y << 16), __uint_as_float(rk.y << 16), part);
    part = fmaf(__uint_as_float(rq.y & 0xffff0000u), __uint_as_float(rk.y & 0xffff0000u), part);
    part = warp_sum(part);
    if (lane == 0) p[cnt * G + g] = c.scale * part;
  }
  // K pass: block b (16 rows) of the stream goes to warp b % NW; every warp steps through every tile so that
  // the ring's barriers see all of them.  Besides the raw scores a warp keeps the softmax statistics of its rows
  // (per head: running maximum, and per lane the sum over its own rows), in the shadow of the stream: the pass
  // between the streams is then a merge of NW pairs per head instead of two sweeps over all scores.
  // A sparse pattern inside the recent window (Section 5.1: heavy hitters combined with the strided / fixed patterns)
  // leaves keys out: logit -inf, probability 0, no score from this step; it needs the slots' positions.
  const int mask_kind = c.mask_kind;
  if (mask_kind != 0 && nstr > 0 && !bar_wait(&sh.aux, 0)) timed_out = true;
  float wm[2] = {-INFINITY, -INFINITY}, wl[2] = {0.f, 0.f};  // heads 2 c4 and 2 c4 + 1
  for (int j = 0; j < nt; ++j) {
    const int s = j & (kStages - 1);
    if (!bar_wait(&sh.full[s], (uint32_t)(j >> kStageShift) & 1u)) timed_out = true;
    const int hb = ((warp - 2 * j) & (kWarps - 1));  // this warp's block of the tile: 0 or 1 (else none)
    if (hb < 2) {
      const unsigned char* kt = ring + (size_t)s * kTileBytes + (size_t)(16 * hb) * kRowBytes;
      float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};  // two chains
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        const uint4 ka = *reinterpret_cast<const uint4*>(kt + gl * kRowBytes + 64 * cc + 16 * c4);
        const uint4 kb = *reinterpret_cast<const uint4*>(kt + (gl + 8) * kRowBytes + 64 * cc + 16 * c4);
        mma_16816(d0, ka.x, kb.x, ka.y, kb.y, qb[cc].x, qb[cc].y);
        mma_16816(d1, ka.z, kb.z, ka.w, kb.w, qb[cc].z, qb[cc].w);
      }
      // lane (gl, c4): rows gl and gl + 8 of the block, heads 2 c4 and 2 c4 + 1 (rows past the end hold stale bytes)
      const int rowA = j * kTileRows + 16 * hb + gl, rowB = rowA + 8;
      // (without the statistics only a pattern needs the -inf: rows past the end are not stored at all)
      bool okA = KSTATS ? rowA < cnt : true, okB = KSTATS ? rowB < cnt : true;
      if (mask_kind != 0) {
        okA = rowA < cnt;
        okB = rowB < cnt;
        okA = okA && key_attended(mask_kind, c.mask_a, c.mask_b, pos_s[okA ? rowA : 0], t, r);
        okB = okB && key_attended(mask_kind, c.mask_a, c.mask_b, pos_s[okB ? rowB : 0], t, r);
      }
      float sc[2][2];  // [row A / B][head 2 c4 / 2 c4 + 1]
      sc[0][0] = okA ? c.scale * (d0[0] + d1[0]) : -INFINITY;
      sc[0][1] = okA ? c.scale * (d0[1] + d1[1]) : -INFINITY;
      sc[1][0] = okB ? c.scale * (d0[2] + d1[2]) : -INFINITY;
      sc[1][1] = okB ? c.scale * (d0[3] + d1[3]) : -INFINITY;
      if constexpr (G == 1) {
        if (c4 == 0) {
          if (rowA < cnt) p[rowA] = sc[0][0];
          if (rowB < cnt) p[rowB] = sc[1][0];
        }
      } else if (2 * c4 < G) {
        if (rowA < cnt) *reinterpret_cast<float2*>(p + rowA * G + 2 * c4) = make_float2(sc[0][0], sc[0][1]);
        if (rowB < cnt) *reinterpret_cast<float2*>(p + rowB * G + 2 * c4) = make_float2(sc[1][0], sc[1][1]);
      }
      if constexpr (KSTATS) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float bm = fmaxf(sc[0][h], sc[1][h]);  // the block's maximum of this head: over the eight row pairs
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 4));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 8));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
        const float nm = fmaxf(wm[h], bm);
        if (nm > -INFINITY) {  // (uniform over the lanes of equal c4)
          wl[h] = wl[h] * expf(wm[h] - nm) + expf(sc[0][h] - nm) + expf(sc[1][h] - nm);  // expf(-inf) = 0
          wm[h] = nm;
        }
      }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.empty[s]);
  }
  if constexpr (KSTATS) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {  // the lanes' sums over the warp's rows
    wl[h] += __shfl_xor_sync(0xffffffffu, wl[h], 4);
    wl[h] += __shfl_xor_sync(0xffffffffu, wl[h], 8);
    wl[h] += __shfl_xor_sync(0xffffffffu, wl[h], 16);
    if (gl == 0 && 2 * c4 + h < G) {
      sh.part_m[warp][2 * c4 + h] = wm[h];
      sh.part_l[warp][2 * c4 + h] = wl[h];
    }
  }
  }
  consumer_sync();
  if constexpr (TOPK) {
    // ---- "Top-K" attention (appendix on the Top-K baseline): keep the c.topk largest logits of the step among the
    // kept entries the pattern allows and the token itself; equal logits: the higher position first.  The key of an
    // entry is (order-preserving bits of its logit, position): keys are distinct, so the topk-th largest one is a
    // threshold; it is found by a most-significant-digit radix select, 8 bits a pass, over the scores in shared
    // memory.  What is below it gets logit -inf: probability 0, no value, no score from this step.
    if (nstr > 0 && !bar_wait(&sh.aux, 0)) timed_out = true;  // the slots' positions
    auto key_of = [&](int x) -> unsigned long long {  // x < cnt: cached row x; x == cnt: the token itself
      const float sx = p[x];
      if (!(sx > -INFINITY)) return 0ull;  // left out by the pattern: below every real key
      unsigned int ub = __float_as_uint(sx);
      ub = (ub & 0x80000000u) ? ~ub : (ub | 0x80000000u);
      return ((unsigned long long)ub << 32) | (unsigned int)(x < cnt ? pos_s[x] : t);
    };
    const int ncand = cnt + 1;
    if (tid == 0) {
      sh.tk_prefix = 0ull;
      sh.tk_remaining = (unsigned int)c.topk;
      sh.tk_count = 0u;
    }
    consumer_sync();
    {
      unsigned int real = 0;
      for (int x = tid; x < ncand; x += kThreads) real += key_of(x) != 0ull ? 1u : 0u;
      real = (unsigned int)warp_sum((float)real);  // (at most 8193 per unit: exact in fp32)
      if (lane == 0) atomicAdd(&sh.tk_count, real);
    }
    consumer_sync();
    unsigned long long thr = 1ull;  // every real key
    if (sh.tk_count > (unsigned int)c.topk) {
      for (int pass = 0; pass < 8; ++pass) {
        const int shift = 56 - 8 * pass;
        for (int i = tid; i < 256; i += kThreads) sh.hist[i] = 0u;
        consumer_sync();
        const unsigned long long prefix = sh.tk_prefix;
        const unsigned long long himask = pass == 0 ? 0ull : (~0ull << (shift + 8));
        for (int x = tid; x < ncand; x += kThreads) {
          const unsigned long long key = key_of(x);
          if (key != 0ull && (key & himask) == prefix) atomicAdd(&sh.hist[(unsigned int)(key >> shift) & 255u], 1u);
        }
        consumer_sync();
        if (warp == 0) {  // the bin that holds the rank still looked for, scanning from the top bin down
          const int rem = (int)sh.tk_remaining;
          int cnts[8], tot = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            cnts[i] = (int)sh.hist[255 - 8 * lane - i];
            tot += cnts[i];
          }
          int incl = tot;
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += y;
          }
          int before = incl - tot;
          if (before < rem && incl >= rem) {  // exactly one lane
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              if (before < rem && before + cnts[i] >= rem) {
                sh.tk_prefix = prefix | ((unsigned long long)(255 - 8 * lane - i) << shift);
                sh.tk_remaining = (unsigned int)(rem - before);
                sh.tk_bin = (unsigned int)cnts[i];
                before = rem;  // done
              } else {
                before += cnts[i];
              }
            }
          }
        }
        consumer_sync();
        // after the four passes over the logit's bits: if every entry that shares the threshold logit is wanted
        // (nearly always: it is the only one), the positions need not be looked at
        if (pass == 3 && sh.tk_bin == sh.tk_remaining) break;
      }
      thr = sh.tk_prefix;
    }
    for (int x = tid; x < ncand; x += kThreads)
      if (key_of(x) < thr) p[x] = -INFINITY;
    consumer_sync();
  }
  if constexpr (!KSTATS) {
    // one sweep over the scores instead: thread (x0, g) = (tid / G, tid % G), online pairs merged by shuffles
    const int g = tid % G;
    float mx = -INFINITY, sum = 0.f;
    for (int x = tid / G; x < cnt; x += kThreads / G) {
      const float sx = p[x * G + g];
      if (sx > -INFINITY) {
        if (sx > mx) {
          sum *= expf(mx - sx);  // expf(-inf) = 0 the first time
          mx = sx;
        }
        sum += expf(sx - mx);
      }
    }
#pragma unroll
    for (int off = G; off < 32; off <<= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, mx, off), os = __shfl_xor_sync(0xffffffffu, sum, off);
      const float nm = fmaxf(mx, om);
      sum = (mx > -INFINITY ? sum * expf(mx - nm) : 0.f) + (om > -INFINITY ? os * expf(om - nm) : 0.f);
      mx = nm;
    }
    if (lane < G) {
      sh.part_m[warp][lane] = mx;
      sh.part_l[warp][lane] = sum;
    }
    consumer_sync();
  }

  // ---- softmax statistics per head: the warps' pairs and the token itself (exact maximum and sum) --------------
  {
    if (tid < G) {
      const float s_self = rank == 0 ? p[cnt * G + tid] : -INFINITY;
      float m = s_self;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) m = fmaxf(m, sh.part_m[w][tid]);
      float l = s_self > -INFINITY ? expf(s_self - m) : 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w)
        if (sh.part_m[w][tid] > -INFINITY) l += sh.part_l[w][tid] * expf(sh.part_m[w][tid] - m);
      sh.m[tid] = m;
      sh.inv_l[tid] = split == 1 ? 1.0f / l : l;  // (split unit: the block's own sum, until the cluster's is known)
    }
    if (split > 1) {
      // the block's statistics into every block of the cluster (its own included); the value tiles keep arriving
      // in the ring meanwhile
      cluster.barrier_wait();  // every peer is running: its shared memory may be written
      consumer_sync();
      if (tid < split * G) {
        const int dst = tid / G, g2 = tid % G;
        *cluster.map_shared_rank(&sh.x_m[rank][g2], dst) = sh.m[g2];
        *cluster.map_shared_rank(&sh.x_l[rank][g2], dst) = sh.inv_l[g2];
      }
      cluster.sync();
      if (tid < G) {
        float m = -INFINITY;
        for (int rk = 0; rk < split; ++rk) m = fmaxf(m, sh.x_m[rk][tid]);
        float l = 0.f;
        for (int rk = 0; rk < split; ++rk)
          if (sh.x_m[rk][tid] > -INFINITY) l += sh.x_l[rk][tid] * expf(sh.x_m[rk][tid] - m);
        sh.m[tid] = m;
        sh.inv_l[tid] = 1.0f / l;
      }
    }
    consumer_sync();
    // final probabilities in place: thread (x0, g) = (tid / G, tid % G); -inf (a key the pattern left out) gives 0
    {
      const int g = tid % G;
      const float m = sh.m[g], inv_l = sh.inv_l[g];
      for (int x = tid / G; x < cnt + (rank == 0 ? 1 : 0); x += kThreads / G) p[x * G + g] = expf(p[x * G + g] - m) * inv_l;
    }
  }
  consumer_sync();

  // ---- V pass: lane = (row of the warp's pair, eight channels); G x 8 accumulators ---------------------------
  const int sub = lane >> 4, ch = lane & 15;
  float o[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int v = 0; v < 8; ++v) o[g][v] = 0.f;
  for (int j = 0; j < nt; ++j) {
    const int T = nt + j, s = T & (kStages - 1);
    if (!bar_wait(&sh.full[s], (uint32_t)(T >> kStageShift) & 1u)) timed_out = true;
    const unsigned char* vt = ring + (size_t)s * kTileBytes;
#pragma unroll
    for (int ps = 0; ps < kTileRows / (2 * kWarps); ++ps) {
      const int rl = ps * 2 * kWarps + 2 * warp + sub, row = j * kTileRows + rl;
      if (row < cnt) {
        float vf[8];
        Vec16<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(vt + rl * kRowBytes + 16 * ch), vf);
        float pr[G];
        if constexpr (G == 1) {
          pr[0] = p[row];
        } else if constexpr (G == 2) {
          const float2 p2 = *reinterpret_cast<const float2*>(p + row * G);
          pr[0] = p2.x;
          pr[1] = p2.y;
        } else {
#pragma unroll
          for (int g4 = 0; g4 < G / 4; ++g4) {
            const float4 p4 = *reinterpret_cast<const float4*>(p + row * G + 4 * g4);
            pr[4 * g4] = p4.x;
            pr[4 * g4 + 1] = p4.y;
            pr[4 * g4 + 2] = p4.z;
            pr[4 * g4 + 3] = p4.w;
          }
        }
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
          for (int v = 0; v < 8; v += 2) {
            const float2 t2 = __ffma2_rn(make_float2(pr[g], pr[g]), make_float2(vf[v], vf[v + 1]), make_float2(o[g][v], o[g][v + 1]));
            o[g][v] = t2.x;
            o[g][v + 1] = t2.y;
          }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.empty[s]);
  }
  // the ring is free once every warp has read its last tile: it takes the partial outputs
  consumer_sync();
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float* dst = red + ((size_t)(2 * warp + sub) * G + g) * kD + 8 * ch;
    *reinterpret_cast<float4*>(dst) = make_float4(o[g][0], o[g][1], o[g][2], o[g][3]);
    *reinterpret_cast<float4*>(dst + 4) = make_float4(o[g][4], o[g][5], o[g][6], o[g][7]);
  }
  // (the staged scores and positions arrived long ago)
  if (nstr > 0 && !bar_wait(&sh.aux, 0)) timed_out = true;
  consumer_sync();
  // the block's partial outputs (normalised by the unit's sums already); rank 0 adds the new token's own value
  for (int i = tid; i < G * kD; i += kThreads) {
    const int g = i / kD, x = i % kD;
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < 2 * kWarps; ++w) acc += red[((size_t)w * G + g) * kD + x];
    if (rank == 0) acc = fmaf(p[cnt * G + g], __bfloat162float(vu[x]), acc);
    if (split == 1) out[((int64_t)u * G + g) * kD + x] = __float2bfloat16_rn(acc);
    else *cluster.map_shared_rank(x_out + ((size_t)rank * G + g) * kD + x, 0) = acc;
  }

  // ---- accumulate (every head's probability), victim, in-place write ----------------------------------------
  const bool full = cnt_u >= B;
  Cand best = cand_none();
  for (int x = tid; x < cnt; x += kThreads) {
    double px = 0.0;
#pragma unroll
    for (int g = 0; g < G; ++g) px += (double)p[x * G + g];
    const double a = acc_s[x] + px;
    if (H2O_IN_RANGE(mt.slot_off + lo + x, c.total_slots, c.status)) acc_g[x] = a;
    const int ps = pos_s[x];
    if (full && ps <= t - r) {
      const double score = c.score_mode == 1 ? a / (double)(t - ps + 1) : a;
      const Cand cx{(unsigned long long)__double_as_longlong(score), ps, lo + x};
      if (cand_before(cx, best)) best = cx;
    }
  }
  double p_self = 0.0;
  if (rank == 0) {
#pragma unroll
    for (int g = 0; g < G; ++g) p_self += (double)p[cnt * G + g];
  }
  if (rank == 0 && tid == 0 && full && r == 0) {  // without a recent window the new token competes too
    const Cand cs{(unsigned long long)__double_as_longlong(p_self), t, -2};
    if (cand_before(cs, best)) best = cs;
  }
  best = warp_argmin(best);
  if (lane == 0) sh.wbest[warp] = best;
  if (timed_out) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
  // the new token's K/V row in 16-byte pieces, fetched before the barrier so that the round trip overlaps it
  uint4 new_row = make_uint4(0, 0, 0, 0);
  if (warp == 0 && rank == 0) new_row = *reinterpret_cast<const uint4*>((lane < 16 ? ku : vu) + (lane & 15) * 8);
  consumer_sync();
  Cand b = cand_none();
  if (warp == 0) b = warp_argmin(lane < kWarps ? sh.wbest[lane] : cand_none());
  if (split > 1) {
    // the block's candidate to rank 0 (its partial outputs went there above); one cluster barrier for both, the
    // last one: afterwards rank 0 works on its own memory only
    if (warp == 0 && lane == 0) *cluster.map_shared_rank(&sh.x_cand[rank], 0) = b;
    cluster.sync();
    if (rank != 0) return;
    for (int i = tid; i < G * kD; i += kThreads) {
      float acc = 0.f;
      for (int rk = 0; rk < split; ++rk) acc += x_out[(size_t)rk * G * kD + i];  // fixed order
      out[(int64_t)u * G * kD + i] = __float2bfloat16_rn(acc);
    }
    if (warp == 0) b = warp_argmin(lane < split ? sh.x_cand[lane] : cand_none());
  }
  if (warp == 0) {
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
    if (slot >= 0 && (!H2O_IN_RANGE(slot, B, c.status) || !H2O_IN_RANGE(mt.slot_off + slot, c.total_slots, c.status))) slot = -1;
    if (lane == 0) {
      if (!full) c.count[su] = cnt_u + 1;
      if (slot >= 0) {
        c.acc[mt.slot_off + slot] = p_self;
        c.pos[mt.slot_off + slot] = t;
      }
      if (evicted_pos) evicted_pos[u] = ev;
      c.tpos[su] = t + 1;
    }
    if (slot >= 0) {  // the new K/V row goes straight into the freed slot
      __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(lane < 16 ? c.K : c.V) + (mt.slot_off + slot) * kD + (lane & 15) * 8;
      *reinterpret_cast<uint4*>(dst) = new_row;
    }
  }
}

size_t ring_smem(int group, int chunk, int stages) {
  return (size_t)stages * kTileBytes + (size_t)chunk * 12 + (size_t)(chunk + 4) * group * sizeof(float);
}

template <int G, int NW, int STAGES, int MINB, bool CLUSTER = false, bool TOPK = false>
cudaError_t launch_ring(const CacheView& c, int split, int chunk, int launch_flags, const void* q, const void* k_new,
                        const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream) {
  constexpr int kStages = STAGES;
  static_assert(STAGES == 4 || STAGES == 8, "ring depth");
  static_assert((size_t)2 * NW * G * kD * sizeof(float) <= (size_t)kStages * kTileBytes, "partial outputs reuse the ring");
  const size_t smem = ring_smem(G, chunk, kStages) + (split > 1 ? (size_t)kMaxSplit * G * kD * sizeof(float) : 0);
  static unsigned long long attr_flags = 0;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_two_pass_kernel<G, NW, STAGES, MINB, CLUSTER, TOPK>), 200 * 1024, &attr_flags);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(c.units * split));
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
  cfg.numAttrs = split > 1 ? 3 : 1;
  return cudaLaunchKernelEx(&cfg, decode_two_pass_kernel<G, NW, STAGES, MINB, CLUSTER, TOPK>, c, static_cast<const __nv_bfloat16*>(q),
                            static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
                            static_cast<__nv_bfloat16*>(out), evicted_pos, split, chunk, launch_flags);
}

template <int G>
cudaError_t launch_ring_g(const CacheView& c, int split, int chunk, int launch_flags, const void* q, const void* k_new,
                          const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream) {
  if (c.topk > 0) {  // "Top-K" attention: multi-head, one block per unit
    if constexpr (G == 1) {
      if (split != 1) return cudaErrorInvalidValue;
      if (c.units <= 2 * sm_count())
        return launch_ring<G, 8, 8, 2, false, true>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
      return launch_ring<G, 4, 4, 4, false, true>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
    } else {
      return cudaErrorInvalidValue;
    }
  }
  if (split > 1) {
    if constexpr (G == 1) {
      if (c.units * split <= 2 * sm_count())
        return launch_ring<G, 8, 8, 2, true>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
      return launch_ring<G, 4, 4, 4, true>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
    } else {
      return cudaErrorInvalidValue;  // grouped caches are not split
    }
  }
  if (c.units <= 2 * sm_count())
    return launch_ring<G, 8, 8, 2>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
  // five blocks per SM (72 registers) where their shared memory allows it: 2048 units of 256 slots 51.1 -> 48.0 us,
  // 3584 units of 104 slots 51.4 -> 45.6 us; with four blocks' worth of shared memory the cap only costs (config 5:
  // 140.5 -> 142.1 us)
  if constexpr (G == 1) {
    if (5 * (ring_smem(G, chunk, 4) + 2048) <= 227 * 1024)
      return launch_ring<G, 4, 4, 5>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
  }
  return launch_ring<G, 4, 4, 4>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
}

}  // namespace

// Does the streaming kernel serve this cache (bf16, head_dim 128, its staging within the shared memory of a block)?
// chunk: slots per thread block (the whole budget, or its share when a unit is split over a cluster).
bool decode_two_pass_supported(int dtype, int head_dim, int group, int chunk) {
  if (dtype != H2O_BF16 || head_dim != kD || (group != 1 && group != 2 && group != 4 && group != 8)) return false;
  return ring_smem(group, (chunk + 3) & ~3, kMaxStages) + (size_t)kMaxSplit * group * kD * sizeof(float) <= 190 * 1024;
}

cudaError_t launch_decode_two_pass(const CacheView& c, int split, int chunk, bool cache_is_quiescent, bool all_full,
                                   const void* q, const void* k_new, const void* v_new, void* out, int32_t* evicted_pos,
                                   cudaStream_t stream) {
  if (split < 1 || split > kMaxSplit || (chunk & 3) != 0) return cudaErrorInvalidValue;
  const int launch_flags = (cache_is_quiescent ? 1 : 0) | (all_full ? 2 : 0);
  switch (c.group) {
    case 1: return launch_ring_g<1>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
    case 2: return launch_ring_g<2>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
    case 4: return launch_ring_g<4>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
    case 8: return launch_ring_g<8>(c, split, chunk, launch_flags, q, k_new, v_new, out, evicted_pos, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace h2o
