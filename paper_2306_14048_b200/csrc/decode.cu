// Fused decode step: scores over the occupied slots, softmax, weighted values,
// score accumulation, victim search and in-place replacement — one kernel launch,
// the cache read exactly once.
//
// Paper: Algorithm 2 loop body (scores, accumulate, argmax of F_score(G \ {v}), which
// for the summation score is the candidate with the smallest accumulated score) on
// the pre-allocated, overwritten-in-place cache of Section 4.2 / Appendix A.
//
// Shape of the kernel (the step is bound by HBM traffic, about one flop per byte):
//   - A unit's slots are split over `split` thread blocks that form one cluster; each
//     block owns `chunk` consecutive slots.  split = 1 for many small units, up to 8
//     for few long ones, so that every SM has several blocks resident.
//   - The slots are streamed as pairs of an 8 KB K tile and the matching 8 KB V tile into a
//     shared-memory ring with cp.async.bulk (the TMA engine, one elected thread issues,
//     completion counted on an mbarrier).  The first STAGES pairs are issued before anything
//     else happens.
//   - Every row group of a warp keeps its own online softmax (running maximum, sum and partial
//     output); the groups are merged once after the stream.  Raw scores stay in shared memory:
//     the final probabilities that are accumulated use the exact maximum and sum.  Blocks of a
//     cluster exchange (max, sum), partial outputs and victim candidates through distributed
//     shared memory.
//   - Accumulated scores are fp64 in memory: eviction decisions compare sums of
//     hundreds of probabilities and must not depend on fp32 rounding of the sum.
// Every wait on an mbarrier is bounded; a wait that gives up records H2O_ERR_TIMEOUT in
// the status word and the block carries on (results of that step are then invalid).
#include <climits>
#include <cooperative_groups.h>

#include "h2o_internal.cuh"

namespace cg = cooperative_groups;

namespace h2o {

namespace {

// Consumer warps per block: 8 by default; 4 for launches of many small units (more blocks resident per
// SM hide one another's serial prologue and epilogue, which dominate a unit of a few tiles).
constexpr int kMaxWarps = 8;
constexpr int kSmallUnitRows = 160;  // largest block share (slots) served by the 4-warp variant
constexpr int kTileBytes = 8192;  // (4 KB tiles with twice the depth and 16 KB tiles with half of it were slower)
constexpr int kMaxStages = 8;
constexpr int kDefaultStages = 4;
constexpr int kMaxSplit = 8;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kMaxDynSmem = 200 * 1024;  // plus ~9 KB static shared memory stays below the 227 KB limit

// Eviction candidate.  Accumulated scores are sums of probabilities (>= 0), so the bit
// pattern of the double orders like its value; comparing the integer key keeps the
// (slow) fp64 pipe out of the search.
struct Cand {
  unsigned long long key;  // bit pattern of the accumulated score
  int pos;
  int slot;  // slot index inside the unit; -1: none, -2: the new token itself
};
__device__ __forceinline__ Cand cand_none() { return Cand{~0ull, INT_MAX, -1}; }
__device__ __forceinline__ Cand cand_make(double acc, int pos, int slot) {
  return Cand{(unsigned long long)__double_as_longlong(acc), pos, slot};
}
__device__ __forceinline__ bool cand_before(const Cand& a, const Cand& b) {
  if (a.slot == -1) return false;
  if (b.slot == -1) return true;
  return a.key < b.key || (a.key == b.key && a.pos < b.pos);
}

// Warp-wide minimum under the eviction order; every lane gets the winner.  Accumulated
// scores are >= 0, so their bit patterns order like the values and three 32-bit
// hardware reductions (high word, low word, position) find the winner.
__device__ __forceinline__ Cand warp_argmin(const Cand& a) {
  const bool valid = a.slot != -1;
  const unsigned long long bits = valid ? a.key : ~0ull;
  const unsigned hi = (unsigned)(bits >> 32), lo = (unsigned)bits;
  const unsigned mh = __reduce_min_sync(0xffffffffu, hi);
  const unsigned ml = __reduce_min_sync(0xffffffffu, hi == mh ? lo : 0xffffffffu);
  const bool tie = valid && hi == mh && lo == ml;
  const unsigned mp = __reduce_min_sync(0xffffffffu, tie ? (unsigned)a.pos : 0xffffffffu);
  const unsigned who = __ballot_sync(0xffffffffu, tie && (unsigned)a.pos == mp);
  if (who == 0) return cand_none();
  const int src = __ffs(who) - 1;
  Cand b;
  b.key = ((unsigned long long)mh << 32) | ml;
  b.pos = (int)mp;
  b.slot = __shfl_sync(0xffffffffu, a.slot, src);
  return b;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false after kSpinLimit unsuccessful polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> shared bulk copy (16-byte aligned addresses, size a multiple of 16)
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// Optional phase timers (compile with -DH2O_PHASE_TIMERS): thread 0 of every block records %globaltimer (ns,
// common to all SMs) at a few points, for the last eight launches (the host numbers the launches in the upper bits
// of launch_flags), and its SM in entry 0; h2o_debug_phase_timers copies them out.  Off in normal builds.
#ifdef H2O_PHASE_TIMERS
constexpr int kPhaseBlocks = 4096, kPhaseLaunches = 8;
__device__ unsigned long long g_phase[kPhaseLaunches * kPhaseBlocks * 16];
#define H2O_STAMP(i)                                                                                        \
  do {                                                                                                      \
    if (threadIdx.x == 0 && blockIdx.x < kPhaseBlocks) {                                                    \
      unsigned long long ts_;                                                                               \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ts_));                                             \
      g_phase[((((unsigned)launch_flags >> 8) % kPhaseLaunches) * kPhaseBlocks + blockIdx.x) * 16 + (i)] = ts_; \
    }                                                                                                       \
  } while (0)
#else
#define H2O_STAMP(i) do { } while (0)
#endif

template <typename T, int D, int NW>
struct Cfg {
  static constexpr int VEC = Vec16<T>::N;
  static constexpr int LPR = D / VEC;                  // lanes per row
  static constexpr int RPW = 32 / LPR;                 // rows per warp pass (= row groups per warp)
  static constexpr int RPC = NW * RPW;                 // rows per block pass
  static constexpr int GROUPS = NW * RPW;              // independent online-softmax streams per block
  static constexpr int ROW_BYTES = D * (int)sizeof(T);
  static constexpr int TILE_ROWS = kTileBytes / ROW_BYTES;
  static constexpr int PASSES = TILE_ROWS / RPC;
  static_assert(TILE_ROWS % RPC == 0 && PASSES >= 1, "tile must be a whole number of block passes");
  static_assert(GROUPS <= 32, "group statistics are combined by one warp");
};

template <int GROUPS, int D>
struct Shared {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t aux;
  float red[GROUPS][D];  // per-group partial outputs (unnormalised, relative to the group's maximum)
  float gm[GROUPS], gl[GROUPS];
  Cand wbest[kMaxWarps];
  // "Top-K" attention: histogram and state of the radix select over the step's logits
  unsigned int hist[256];
  unsigned long long tk_prefix;
  unsigned int tk_remaining, tk_count, tk_bin;  // tk_bin: entries in the bin the last pass chose
  // Cluster exchange: every block PUSHES its values into its peers' shared memory (remote stores are
  // fire-and-forget, remote loads a round trip), then one cluster barrier makes them visible.
  float x_m[kMaxSplit], x_l[kMaxSplit];  // block statistics of every rank (written by that rank)
  Cand x_cand[kMaxSplit];                // rank 0 only: every rank's eviction candidate
  // (the partial outputs pushed to rank 0, [kMaxSplit][D] floats, live in dynamic shared memory and
  //  exist only in launches that split a unit, so that unsplit launches keep their blocks per SM)
};

template <int THREADS>
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory"); }

// MINB is the number of blocks per SM the register allocation must leave room for.  A launch with at
// most two blocks per SM runs fastest with all the registers the compiler wants (MINB 1: no spills, more
// loads in flight per thread); a launch with many blocks per SM is bound by how many of them are
// resident to hide one another's serial prologue and epilogue (MINB 4).
// TOPK: the instance with "Top-K" attention (its selection code costs registers the plain step must not pay for).
template <typename T, int D, int MINB, int NW, bool TOPK>
__global__ void __launch_bounds__(NW * 32 + 32, MINB)
decode_kernel(CacheView c, const T* __restrict__ q, const T* __restrict__ k_new, const T* __restrict__ v_new,
              T* __restrict__ out, int32_t* __restrict__ evicted_pos, int split, int chunk, int stages, int stage_shift,
              int launch_flags) {
  // stages = 1 << stage_shift, the ring depth: a power of two, so that slot and phase of tile j are a mask and a
  // shift.  The register-capped instances (MINB >= 4) keep the division by the run-time depth: there the cheaper
  // form changed the register allocation into spilling and was slower (3584 units of 104 slots: 44.2 -> 47.0 us),
  // in the uncapped instance it is faster (256 units of 410 slots: 12.7 -> 12.2 us).
  auto ring_slot = [&](int j) { return MINB >= 4 ? j % stages : (j & (stages - 1)); };
  auto ring_turn = [&](int j) { return MINB >= 4 ? j / stages : (j >> stage_shift); };
  using C = Cfg<T, D, NW>;
  constexpr int kWarps = NW, kThreads = NW * 32;
  constexpr int VEC = C::VEC, LPR = C::LPR, RPW = C::RPW, RPC = C::RPC, TILE_ROWS = C::TILE_ROWS, GROUPS = C::GROUPS;
  extern __shared__ __align__(128) unsigned char dyn[];
  __shared__ Shared<GROUPS, D> sh;
  // dynamic layout: ring[stages][K tile | V tile] | acc_s[chunk] f64 | pos_s[chunk] i32 | p[chunk + 1] f32
  unsigned char* ring = dyn;
  double* acc_s = reinterpret_cast<double*>(dyn + (size_t)stages * 2 * kTileBytes);
  int32_t* pos_s = reinterpret_cast<int32_t*>(acc_s + chunk);
  float* p = reinterpret_cast<float*>(pos_s + chunk);
  float* x_out = p + chunk + 4;  // [kMaxSplit][D], only when split > 1 (behind the 16 spare bytes of p)

  H2O_STAMP(1);
#ifdef H2O_PHASE_TIMERS
  if (threadIdx.x == 0 && blockIdx.x < kPhaseBlocks) {
    unsigned smid_;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid_));
    g_phase[((((unsigned)launch_flags >> 8) % kPhaseLaunches) * kPhaseBlocks + blockIdx.x) * 16 + 0] = smid_;
  }
#endif
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPR, ch = lane % LPR;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = split > 1 ? (int)cluster.block_rank() : 0;
  // Early arrival on the cluster barrier; the matching wait comes right before the first remote
  // store, by which time every block of the cluster has long started (its shared memory exists).
  if (split > 1) cluster.barrier_arrive();
  const int su = blockIdx.x / split;  // launch position of the unit
  const bool cache_is_quiescent = (launch_flags & 1) != 0, all_full = (launch_flags & 2) != 0;
  // the unit's static description: arithmetic when all budgets are equal, else one load from the table
  // written at create time
  UnitMeta mt;
  if (c.uni_pad >= 0) {
    mt.slot_off = (int64_t)su * c.uni_pad;
    mt.unit = su;
    mt.kbud = c.uni_k;
    mt.rwin = c.uni_r;
    mt.pad_ = 0;
  } else {
    mt = c.meta[su];
  }
  // Programmatic dependent launch: this grid may have been started while the previous kernel of
  // the stream was still running.  What it may touch before that kernel has finished
  // (griddepcontrol.wait) depends on who wrote what:
  //   - q / k_new / v_new can come from any kernel, so they are read only after the wait;
  //   - the cache itself is written by this library alone.  The host tells us whether its previous
  //     launch on this stream could have written THIS cache; if not (`cache_is_quiescent`), the cache
  //     tiles are prefetched into shared memory before the wait, which hides the start-up latency.
  // The next grid is released (launch_dependents) only after this grid's own wait: when a grid
  // starts, everything older than its immediate predecessor has therefore completed.
  if (!cache_is_quiescent) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  const int u = mt.unit, r = mt.rwin, B = mt.kbud + mt.rwin;
  const int lo = rank * chunk;                            // first slot of this block
  // How many slots to stream.  Normally the occupied ones, which takes the counter from memory first.
  // When the host expects every unit to be full (`all_full`) the block streams its whole share of the
  // budget at once and reads the counter meanwhile: with equal budgets the first copies then depend on
  // no load at all.  The expectation only decides WHAT IS FETCHED — rows beyond the real count are
  // never used — so a stale flag (say, in a replayed CUDA graph) costs bandwidth, not correctness.
  int cnt = 0;
  if (!all_full) cnt = c.count[su];
  int nstr = all_full ? max(0, min(B - lo, chunk)) : max(0, min(cnt - lo, chunk));
  // (checked build: the unit and the whole range of rows this block streams must lie inside the cache)
  if (!H2O_IN_RANGE(mt.unit, c.units, c.status) ||
      (nstr > 0 && !H2O_IN_RANGE(mt.slot_off + lo + ((nstr + 3) & ~3) - 1, c.total_slots, c.status)))
    nstr = 0;
  const int ntile = (nstr + TILE_ROWS - 1) / TILE_ROWS;   // stages to stream (one K tile + one V tile each)
  T* Kb = reinterpret_cast<T*>(c.K) + (mt.slot_off + lo) * D;
  T* Vb = reinterpret_cast<T*>(c.V) + (mt.slot_off + lo) * D;
  double* acc_g = c.acc + mt.slot_off + lo;
  int32_t* pos_g = c.pos + mt.slot_off + lo;
  const T* qu = q + (int64_t)u * D;
  const T* ku = k_new + (int64_t)u * D;
  const T* vu = v_new + (int64_t)u * D;
  bool timed_out = false;

  auto issue_stage = [&](int j) {  // producer lane only
    const int s = ring_slot(j);
    const int rows = min(TILE_ROWS, nstr - j * TILE_ROWS);
    const uint32_t bytes = (uint32_t)rows * C::ROW_BYTES;
    unsigned char* dst = ring + (size_t)s * 2 * kTileBytes;
    // ("Top-K" attention streams the keys only: which value rows are needed is known after the last score)
    mbar_expect_tx(&sh.full[s], TOPK ? bytes : 2 * bytes);
    bulk_g2s(dst, Kb + (int64_t)j * TILE_ROWS * D, bytes, &sh.full[s]);
    if (!TOPK) bulk_g2s(dst + kTileBytes, Vb + (int64_t)j * TILE_ROWS * D, bytes, &sh.full[s]);
  };
  if (tid == kThreads) {  // producer lane: set up the barriers and get the first tiles moving at once
    for (int s = 0; s < stages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], kWarps);
    }
    mbar_init(&sh.aux, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int j = 0; j < min(stages, ntile); ++j) issue_stage(j);
    if (nstr > 0) {
      const int npad = (nstr + 3) & ~3;  // stays inside the unit's padded slot range
      mbar_expect_tx(&sh.aux, (uint32_t)npad * 12u);
      bulk_g2s(acc_s, acc_g, (uint32_t)npad * 8u, &sh.aux);
      bulk_g2s(pos_s, pos_g, (uint32_t)npad * 4u, &sh.aux);
    }
  }
  if (all_full) cnt = c.count[su];
  if (!H2O_IN_RANGE(cnt, B + 1, c.status)) cnt = 0;  // (checked build) a unit never holds more than its budget
  const int t = c.tpos[su];
  const int nloc = max(0, min(min(cnt - lo, chunk), nstr));  // occupied slots of this block
  __syncthreads();  // barriers are initialised before any consumer polls them
  H2O_STAMP(12);
  if (cache_is_quiescent) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  H2O_STAMP(13);

  // the new token's own key/value: loaded now, used after the stream
  float qf[VEC], ksf[VEC], vself = 0.f;
  Vec16<T>::load(qu + ch * VEC, qf);
  Vec16<T>::load(ku + ch * VEC, ksf);
  if (tid < D) {
    if constexpr (sizeof(T) == 4) vself = *reinterpret_cast<const float*>(vu + tid);
    else vself = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vu + tid));
  }
  float m = 0.f, l = 1.f, s_self = -INFINITY;

  if (warp == kWarps) {
    // ---- producer warp: one lane streams the tiles through the ring ------------------
    if (lane == 0) {
      for (int j = stages; j < ntile; ++j) {
        if (!mbar_wait(&sh.empty[ring_slot(j)], (uint32_t)(ring_turn(j) - 1) & 1u)) timed_out = true;
        issue_stage(j);
      }
    }
    if (timed_out) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
    __syncwarp();
    if (split > 1) {  // the producer warp only keeps the cluster barriers balanced
      cluster.barrier_wait();
      cluster.sync();
      cluster.sync();
    }
  } else {
    // ---- consumer warps: every row group keeps its own online softmax ------------------
    float o[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) o[v] = 0.f;
    float mg = -INFINITY, lg = 0.f;
    {  // score of the new token against itself (every warp computes the same value)
      float part = 0.f;
#pragma unroll
      for (int v = 0; v < VEC; ++v) part = fmaf(qf[v], ksf[v], part);
#pragma unroll
      for (int off = LPR / 2; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
      s_self = c.scale * __shfl_sync(0xffffffffu, part, 0);
    }
    // a sparse pattern needs the slots' positions during the stream (they are staged with the scores)
    const int mask_kind = c.mask_kind;
    constexpr bool topk_mode = TOPK;  // (the host launches one block per unit then: split == 1)
    if (mask_kind != 0 && nloc > 0 && !mbar_wait(&sh.aux, 0)) timed_out = true;
    for (int j = 0; j < ntile; ++j) {
      const int s = ring_slot(j);
      if (!mbar_wait(&sh.full[s], (uint32_t)ring_turn(j) & 1u)) timed_out = true;
      if (j == 0) H2O_STAMP(2);
      const T* kt = reinterpret_cast<const T*>(ring + (size_t)s * 2 * kTileBytes);
      const T* vt = reinterpret_cast<const T*>(ring + (size_t)s * 2 * kTileBytes + kTileBytes);
      const int rows = min(TILE_ROWS, nloc - j * TILE_ROWS);
      float sc[C::PASSES], vf[C::PASSES][VEC];
#pragma unroll
      for (int ps = 0; ps < C::PASSES; ++ps) {  // independent dot products first
        const int row = ps * RPC + warp * RPW + sub;
        float part = 0.f;
        if (row < rows) {
          float kf[VEC];
          Vec16<T>::load(kt + row * D + ch * VEC, kf);
          if (!topk_mode) Vec16<T>::load(vt + row * D + ch * VEC, vf[ps]);
          float2 d2 = make_float2(0.f, 0.f);  // two fp32 FMAs per instruction (packed fp32x2 of this architecture)
#pragma unroll
          for (int v = 0; v < VEC; v += 2)
            d2 = __ffma2_rn(make_float2(qf[v], qf[v + 1]), make_float2(kf[v], kf[v + 1]), d2);
          part = d2.x + d2.y;
        } else {
#pragma unroll
          for (int v = 0; v < VEC; ++v) vf[ps][v] = 0.f;
        }
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        sc[ps] = row < rows ? c.scale * part : -INFINITY;
        if (mask_kind != 0 && row < rows && !key_attended(mask_kind, c.mask_a, c.mask_b, pos_s[j * TILE_ROWS + row], t, r))
          sc[ps] = -INFINITY;  // left out by the pattern: probability 0, no score from this step
        if (ch == 0 && row < rows) p[j * TILE_ROWS + row] = sc[ps];  // raw score, finalised after the stream
      }
      float mnew = mg;
#pragma unroll
      for (int ps = 0; ps < C::PASSES; ++ps) mnew = fmaxf(mnew, sc[ps]);
      if (topk_mode) mnew = -INFINITY;  // scores only: softmax and values follow the selection
      if (mnew > -INFINITY) {  // at least one real row so far in this group
        const float f = expf(mg - mnew);  // expf(-inf) = 0 for the group's first rows
        lg *= f;
#pragma unroll
        for (int v = 0; v < VEC; v += 2) {
          const float2 t2 = __fmul2_rn(make_float2(o[v], o[v + 1]), make_float2(f, f));
          o[v] = t2.x;
          o[v + 1] = t2.y;
        }
#pragma unroll
        for (int ps = 0; ps < C::PASSES; ++ps) {
          const float e = expf(sc[ps] - mnew);  // 0 for rows past the end
          lg += e;
#pragma unroll
          for (int v = 0; v < VEC; v += 2) {
            const float2 t2 = __ffma2_rn(make_float2(e, e), make_float2(vf[ps][v], vf[ps][v + 1]), make_float2(o[v], o[v + 1]));
            o[v] = t2.x;
            o[v + 1] = t2.y;
          }
        }
        mg = mnew;
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&sh.empty[s])) : "memory");
    }
    H2O_STAMP(3);
    const int g = warp * RPW + sub;
    // (the staged scores and positions arrived long ago; looking at their barrier here instead of after the
    //  statistics takes the barrier operation's latency out of the serial tail)
    if (nloc > 0 && !mbar_wait(&sh.aux, 0)) timed_out = true;
#pragma unroll
    for (int v = 0; v < VEC; ++v) sh.red[g][ch * VEC + v] = o[v];
    if (ch == 0) {
      sh.gm[g] = mg;
      sh.gl[g] = lg;
    }
    consumer_sync<kThreads>();
    {
    H2O_STAMP(8);

    float part_o = 0.f;  // block partial output relative to the block maximum
    if constexpr (TOPK) {
      // ---- "Top-K" attention: keep the c.topk largest logits of the step (the kept entries the pattern allows,
      // and the token itself; equal logits: the higher position first).  All raw scores are in shared memory.
      // The key of an entry is (order-preserving bits of its logit, position): keys are distinct, so the
      // topk-th largest one is a threshold; it is found by a most-significant-digit radix select, 8 bits a pass.
      auto key_of = [&](int x) -> unsigned long long {  // x < nloc: cached row x; x == nloc: the token itself
        const float sx = x < nloc ? p[x] : s_self;
        if (!(sx > -INFINITY)) return 0ull;  // left out by the pattern: below every real key
        unsigned int ub = __float_as_uint(sx);
        ub = (ub & 0x80000000u) ? ~ub : (ub | 0x80000000u);
        return ((unsigned long long)ub << 32) | (unsigned int)(x < nloc ? pos_s[x] : t);
      };
      const int ncand = nloc + 1;
      if (tid == 0) {
        sh.tk_prefix = 0ull;
        sh.tk_remaining = (unsigned int)c.topk;
        sh.tk_count = 0u;
      }
      consumer_sync<kThreads>();
      {
        unsigned int real = 0;
        for (int x = tid; x < ncand; x += kThreads) real += key_of(x) != 0ull ? 1u : 0u;
        real = (unsigned int)warp_sum((float)real);  // (at most 8193 per unit: exact in fp32)
        if (lane == 0) atomicAdd(&sh.tk_count, real);
      }
      consumer_sync<kThreads>();
      unsigned long long thr = 1ull;  // every real key
      if (sh.tk_count > (unsigned int)c.topk) {
        for (int pass = 0; pass < 8; ++pass) {
          const int shift = 56 - 8 * pass;
          for (int i = tid; i < 256; i += kThreads) sh.hist[i] = 0u;
          consumer_sync<kThreads>();
          const unsigned long long prefix = sh.tk_prefix;
          const unsigned long long himask = pass == 0 ? 0ull : (~0ull << (shift + 8));
          for (int x = tid; x < ncand; x += kThreads) {
            const unsigned long long key = key_of(x);
            if (key != 0ull && (key & himask) == prefix) atomicAdd(&sh.hist[(unsigned int)(key >> shift) & 255u], 1u);
          }
          consumer_sync<kThreads>();
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
          consumer_sync<kThreads>();
          // after the four passes over the logit's bits: if every entry that shares the threshold logit is wanted
          // (nearly always: it is the only one), the positions need not be looked at
          if (pass == 3 && sh.tk_bin == sh.tk_remaining) break;
        }
        thr = sh.tk_prefix;
      }
      // drop what is below the threshold; block statistics over what is left
      if (key_of(nloc) < thr) s_self = -INFINITY;  // (every thread alike)
      float mx = -INFINITY;
      for (int x = tid; x < nloc; x += kThreads) {
        if (key_of(x) < thr) p[x] = -INFINITY;
        mx = fmaxf(mx, p[x]);
      }
      mx = warp_max(mx);
      if (lane == 0) sh.gm[warp] = mx;
      consumer_sync<kThreads>();
      float mc = s_self;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) mc = fmaxf(mc, sh.gm[w]);
      float sum = 0.f;
      for (int x = tid; x < nloc; x += kThreads) sum += p[x] > -INFINITY ? expf(p[x] - mc) : 0.f;
      sum = warp_sum(sum);
      if (lane == 0) sh.gl[warp] = sum;
      // the value rows of the attended entries, straight from memory (row group g takes rows g, g + GROUPS, ...)
      float ov[VEC];
#pragma unroll
      for (int v = 0; v < VEC; ++v) ov[v] = 0.f;
      for (int x = g; x < nloc; x += GROUPS) {
        const float sx = p[x];
        if (sx > -INFINITY) {
          const float ex = expf(sx - mc);
          float vrow[VEC];
          Vec16<T>::load(Vb + (int64_t)x * D + ch * VEC, vrow);
#pragma unroll
          for (int v = 0; v < VEC; ++v) ov[v] = fmaf(ex, vrow[v], ov[v]);
        }
      }
#pragma unroll
      for (int v = 0; v < VEC; ++v) sh.red[g][ch * VEC + v] = ov[v];
      consumer_sync<kThreads>();
      const float w_self = s_self > -INFINITY ? expf(s_self - mc) : 0.f;
      float lc = w_self;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) lc += sh.gl[w];
      if (tid < D) {
#pragma unroll
        for (int g2 = 0; g2 < GROUPS; ++g2) part_o += sh.red[g2][tid];
        part_o = fmaf(w_self, vself, part_o);
      }
      m = mc;
      l = lc;
    } else {
    // ---- block statistics, computed by every warp alike (fixed order, same result) -------
    const float m_i = lane < GROUPS ? sh.gm[lane] : -INFINITY;
    float mc = warp_max(m_i);
    if (rank == 0) mc = fmaxf(mc, s_self);
    // weight of group `lane` relative to the block maximum (0 for empty groups and for an empty block)
    const float w_i = (lane < GROUPS && m_i > -INFINITY) ? expf(m_i - mc) : 0.f;
    float lc = warp_sum(lane < GROUPS ? sh.gl[lane] * w_i : 0.f);
    const float w_self = rank == 0 ? expf(s_self - mc) : 0.f;
    lc += w_self;
    H2O_STAMP(9);
#pragma unroll
    for (int g2 = 0; g2 < GROUPS; ++g2) {
      const float w = __shfl_sync(0xffffffffu, w_i, g2);
      if (tid < D) part_o = fmaf(sh.red[g2][tid], w, part_o);
    }
    part_o = fmaf(w_self, vself, part_o);
    if (split > 1) {
      cluster.barrier_wait();  // every peer is running: its shared memory may be written
      if (tid < split) {       // my statistics into every block of the cluster (my own included)
        *cluster.map_shared_rank(&sh.x_m[rank], tid) = mc;
        *cluster.map_shared_rank(&sh.x_l[rank], tid) = lc;
      }
      if (tid < D) *cluster.map_shared_rank(x_out + rank * D + tid, 0) = part_o;
      cluster.sync();
      const float mr = lane < split ? sh.x_m[lane] : -INFINITY;
      const float lr = lane < split ? sh.x_l[lane] : 0.f;
      m = warp_max(mr);
      l = warp_sum(mr > -INFINITY ? lr * expf(mr - m) : 0.f);
      if (rank == 0 && tid < D) {
        part_o *= expf(mc - m);
        for (int rk = 1; rk < split; ++rk) {
          const float mrk = sh.x_m[rk];
          if (mrk > -INFINITY) part_o = fmaf(x_out[rk * D + tid], expf(mrk - m), part_o);
        }
      }
    } else {
      m = mc;
      l = lc;
    }
    }  // (not "Top-K")
    H2O_STAMP(4);
    const float inv_l = 1.0f / l;
    if (rank == 0 && tid < D) {
      const float res = part_o * inv_l;
      if constexpr (sizeof(T) == 4) reinterpret_cast<float*>(out)[(int64_t)u * D + tid] = res;
      else reinterpret_cast<__nv_bfloat16*>(out)[(int64_t)u * D + tid] = __float2bfloat16_rn(res);
    }

    // ---- final probabilities, accumulation (Algorithm 2: o~_i = o~_{i-1} + o_i), victim search ----
    const bool full = cnt >= B;
    const float p_self = expf(s_self - m) * inv_l;
    Cand best = cand_none();
#pragma unroll 2
    for (int x = tid; x < nloc; x += kThreads) {
      const float px = expf(p[x] - m) * inv_l;
      const double a = acc_s[x] + (double)px;
      if (H2O_IN_RANGE(mt.slot_off + lo + x, c.total_slots, c.status)) acc_g[x] = a;
      const int ps = pos_s[x];
      if (full && ps <= t - r) {
        // averaged variant: the key has been attended by the queries at positions ps .. t
        const Cand cx = cand_make(c.score_mode == 1 ? a / (double)(t - ps + 1) : a, ps, lo + x);
        if (cand_before(cx, best)) best = cx;
      }
    }
    if (rank == 0 && tid == 0 && full && r == 0) {  // without a recent window the new token competes too
      const Cand cs = cand_make((double)p_self, t, -2);  // attended once: its average is its score
      if (cand_before(cs, best)) best = cs;
    }
    H2O_STAMP(10);
    best = warp_argmin(best);
    H2O_STAMP(11);
    if (lane == 0) sh.wbest[warp] = best;
    if (timed_out) atomicCAS(c.status, 0, H2O_ERR_TIMEOUT);
    // The new token's K/V row in 16-byte chunks, for the write into the freed slot at the very end: fetched
    // here (they are in L2 since the start of the kernel) so that the round trip overlaps the barrier and
    // the final reduction instead of following them.
    constexpr int kNewChunks = (2 * LPR + 31) / 32;
    uint4 new_row[kNewChunks];
    if (warp == 0 && rank == 0) {
#pragma unroll
      for (int i2 = 0; i2 < kNewChunks; ++i2) {
        const int i = lane + 32 * i2;
        if (i < 2 * LPR) new_row[i2] = *reinterpret_cast<const uint4*>((i < LPR ? ku : vu) + (i % LPR) * VEC);
      }
    }
    consumer_sync<kThreads>();
    H2O_STAMP(5);
    if (warp == 0) {
      Cand b = warp_argmin(lane < kWarps ? sh.wbest[lane] : cand_none());
      H2O_STAMP(7);
      if (split > 1) {
        if (lane == 0) *cluster.map_shared_rank(&sh.x_cand[rank], 0) = b;
        cluster.sync();  // the last cluster barrier: afterwards rank 0 works on its own memory only
        if (rank == 0) b = warp_argmin(lane < split ? sh.x_cand[lane] : cand_none());
      }
      if (rank == 0) {  // replace the victim in place (or append while the cache is filling)
        int slot, ev;
        if (!full) {
          slot = cnt;
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
          if (!full) c.count[su] = cnt + 1;
          if (slot >= 0) {
            c.acc[mt.slot_off + slot] = (double)p_self;
            c.pos[mt.slot_off + slot] = t;
          }
          if (evicted_pos) evicted_pos[u] = ev;
          c.tpos[su] = t + 1;
        }
        if (slot >= 0) {
#pragma unroll
          for (int i2 = 0; i2 < kNewChunks; ++i2) {  // the new K/V row goes straight into the freed slot
            const int i = lane + 32 * i2;
            if (i < 2 * LPR) {
              T* base = reinterpret_cast<T*>(i < LPR ? c.K : c.V) + (mt.slot_off + slot) * D;
              *reinterpret_cast<uint4*>(base + (i % LPR) * VEC) = new_row[i2];
            }
          }
        }
      }
    } else if (split > 1) {
      cluster.sync();
    }
    }  // epilogue scope
  }
  H2O_STAMP(6);
}

template <typename T, int D, int MINB, int NW, bool TOPK = false>
cudaError_t launch_minb(const CacheView& c, int split, int chunk, int stages_req, int launch_flags, const void* q,
                        const void* k_new, const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream) {
  using C = Cfg<T, D, NW>;
  // Ring depth.  With few blocks (at most two per SM) each block needs a deep ring to keep enough
  // bytes in flight; with many blocks a shallow ring lets more of them be resident, which hides each
  // block's serial prologue and epilogue behind the others' streams.
  const int blocks = c.units * split;
  const int auto_stages = blocks > 4 * sm_count() ? 2 : kDefaultStages;
  const int want = stages_req > 0 ? (stages_req > kMaxStages ? kMaxStages : stages_req) : auto_stages;
  int stages = (chunk + C::TILE_ROWS - 1) / C::TILE_ROWS;
  stages = stages < 1 ? 1 : (stages > want ? want : stages);
  int stage_shift = 0;
  while ((2 << stage_shift) <= stages) ++stage_shift;
  stages = 1 << stage_shift;  // the largest power of two within the wanted depth
  const size_t smem = (size_t)stages * 2 * kTileBytes + (size_t)chunk * 16 + 16 +
                      (split > 1 ? (size_t)kMaxSplit * D * sizeof(float) : 0);
  static unsigned long long attr_flags = 0;  // one word per template instance, one bit per device
  {
    cudaError_t e =
        ensure_dynamic_smem(reinterpret_cast<const void*>(decode_kernel<T, D, MINB, NW, TOPK>), kMaxDynSmem, &attr_flags);
    if (e != cudaSuccess) return e;
  }
  if (smem > (size_t)kMaxDynSmem) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(c.units * split));
  cfg.blockDim = dim3(NW * 32 + 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute at[3];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)split;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  at[2].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
  at[2].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicyLoadBalancing;
  cfg.attrs = at;
  cfg.numAttrs = split > 1 ? 3 : 2;
  return cudaLaunchKernelEx(&cfg, decode_kernel<T, D, MINB, NW, TOPK>, c, static_cast<const T*>(q),
                            static_cast<const T*>(k_new), static_cast<const T*>(v_new), static_cast<T*>(out),
                            evicted_pos, split, chunk, stages, stage_shift, launch_flags);
}

template <typename T, int D>
cudaError_t launch(const CacheView& c, int split, int chunk, int stages_req, int quiescent, const void* q,
                   const void* k_new, const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream) {
  const int blocks = c.units * split;
  if (c.topk > 0)  // "Top-K" attention: its own instance (four blocks per SM; one block per unit)
    return launch_minb<T, D, 4, 8, true>(c, split, chunk, stages_req, quiescent, q, k_new, v_new, out, evicted_pos, stream);
  if (blocks > 4 * sm_count() && chunk <= kSmallUnitRows)  // many small units: half-size blocks, five per SM
    return launch_minb<T, D, 5, 4>(c, split, chunk, stages_req, quiescent, q, k_new, v_new, out, evicted_pos, stream);
  if (blocks > 2 * sm_count())
    return launch_minb<T, D, 4, 8>(c, split, chunk, stages_req, quiescent, q, k_new, v_new, out, evicted_pos, stream);
  return launch_minb<T, D, 1, 8>(c, split, chunk, stages_req, quiescent, q, k_new, v_new, out, evicted_pos, stream);
}

}  // namespace

#ifdef H2O_PHASE_TIMERS
extern "C" int h2o_debug_phase_timers(unsigned long long* host, int n) {
  return (int)cudaMemcpyFromSymbol(host, g_phase, sizeof(unsigned long long) * (size_t)n);
}
#endif

cudaError_t launch_decode(const CacheView& c, int dtype, int split, int chunk, int stages, bool quiescent_b, bool all_full,
                          const void* q, const void* k_new, const void* v_new, void* out, int32_t* evicted_pos,
                          cudaStream_t stream) {
  if (split < 1 || split > kMaxSplit) return cudaErrorInvalidValue;
  if (c.topk > 0 && split != 1) return cudaErrorInvalidValue;  // the selection runs over one block's scores
  int quiescent = (quiescent_b ? 1 : 0) | (all_full ? 2 : 0);  // launch flags
#ifdef H2O_PHASE_TIMERS
  static int launch_no = 0;
  quiescent |= (launch_no++ & 0xffff) << 8;
#endif
  if (dtype == H2O_F32) {
    if (c.head_dim == 64)
      return launch<float, 64>(c, split, chunk, stages, quiescent, q, k_new, v_new, out, evicted_pos, stream);
    return launch<float, 128>(c, split, chunk, stages, quiescent, q, k_new, v_new, out, evicted_pos, stream);
  }
  if (c.head_dim == 64)
    return launch<__nv_bfloat16, 64>(c, split, chunk, stages, quiescent, q, k_new, v_new, out, evicted_pos, stream);
  return launch<__nv_bfloat16, 128>(c, split, chunk, stages, quiescent, q, k_new, v_new, out, evicted_pos, stream);
}

}  // namespace h2o
