// Prefill selection and gather, one thread block per (sequence, head).
//
// Keep the last r positions and, of positions [0, n - r), the k with the largest
// accumulated score; equal scores are ordered by position (the higher position is
// the stronger one, so that selection equals evicting the weakest candidate
// |C| - k times).  Then copy the kept K/V rows, scores and positions into the
// unit's slots in ascending position order.
//
// The k-th largest score is found with a most-significant-digit radix select on the
// 64-bit pattern of the (non-negative) double scores: 8 passes of 8 bits, one shared
// histogram per pass, the histogram searched by a block-wide scan.  Everything is integer work after the column sums exist, so
// the result is exact.
//
// Paper: Appendix A pseudocode, prefill branch (K heavy hitters and K recent tokens are
// kept; all tokens when the prompt is not longer than 2K).
#include "h2o_internal.cuh"

namespace h2o {

namespace {

constexpr int kSelThreads = 256;

// Ranking key of key j of a prompt of n tokens: its column sum, or (averaged variant) the column sum over
// the number of queries that attended it, n - j.  Both are >= 0, for which the bit pattern is monotone.
__device__ __forceinline__ uint64_t score_key(double a, int j, int n, int mode) {
  if (mode == 1) a = a / (double)(n - j);
  return (uint64_t)__double_as_longlong(a < 0.0 ? 0.0 : a);
}

// Exclusive prefix sum of one int per thread over the block, plus the block total.
__device__ __forceinline__ int block_exclusive_scan(int x, int* warp_tot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = x;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += y;
  }
  __syncthreads();
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int before = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kSelThreads / 32; ++w) {
    const int v = warp_tot[w];
    if (w < warp) before += v;
    tot += v;
  }
  total = tot;
  return before + incl - x;
}

// KPT: candidates' keys a thread holds in registers (0: none, every pass reads them from memory)
template <typename T, int D, int KPT>
__global__ void __launch_bounds__(kSelThreads)
select_gather_kernel(CacheView c, PrefillScratch s, const T* __restrict__ k, const T* __restrict__ v) {
  constexpr int VEC = Vec16<T>::N, LPR = D / VEC;
  extern __shared__ int32_t kept[];  // [min(B, longest prompt)]
  __shared__ unsigned int hist[256];
  __shared__ int warp_tot[kSelThreads / 32];
  __shared__ uint64_t prefix_sh;
  __shared__ int remaining_sh;

  const int tid = threadIdx.x;
  const int su = blockIdx.x;  // launch position
  const UnitMeta mt = c.meta[su];
  const int u = mt.unit;
  const int seq = u / c.n_heads, h = u % c.n_heads;
  const int lo = s.cu[seq], n = s.cu[seq + 1] - lo;
  const int kb = mt.kbud, r = mt.rwin, B = kb + r;
  const double* acc0 = s.acc0 + (int64_t)h * s.total_tokens + lo;
  const int m = n <= B ? n : B;  // entries kept

  if (n <= B) {
    for (int x = tid; x < n; x += kSelThreads) kept[x] = x;
  } else {
    const int nc = n - r;  // candidates [0, nc), nc > kb
    uint64_t thr = 0;      // key of the kb-th largest candidate
    int need_eq = 0;       // how many candidates with key == thr are kept
    int total_eq = 0;
    // The eight radix passes and the count of equal keys all read every candidate's key: up to KPT * 256
    // candidates they are kept in registers (one trip to memory, one division in the averaged mode);
    // longer prompts read them again in every pass.  (KPT follows the longest prompt of the call.)
    const bool cached = KPT > 0 && nc <= kSelThreads * KPT;
    uint64_t keys[KPT > 0 ? KPT : 1];
    if (cached && kb > 0) {
#pragma unroll
      for (int i = 0; i < KPT; ++i) {
        const int j = tid + i * kSelThreads;
        keys[i] = j < nc ? score_key(acc0[j], j, n, c.score_mode) : 0ull;
      }
    }
    auto for_each_key = [&](auto&& f) {
      if (cached) {
#pragma unroll
        for (int i = 0; i < KPT; ++i)
          if (tid + i * kSelThreads < nc) f(keys[i]);
      } else {
        for (int j = tid; j < nc; j += kSelThreads) f(score_key(acc0[j], j, n, c.score_mode));
      }
    };
    if (kb > 0) {
      if (tid == 0) {
        prefix_sh = 0;
        remaining_sh = kb;
      }
      __syncthreads();
      for (int pass = 0; pass < 8; ++pass) {
        const int shift = 56 - 8 * pass;
        hist[tid] = 0;  // kSelThreads == 256 bins
        __syncthreads();
        const uint64_t prefix = prefix_sh;
        const uint64_t himask = pass == 0 ? 0ull : (~0ull << (shift + 8));
        for_each_key([&](uint64_t key) {
          if ((key & himask) == prefix) atomicAdd(&hist[(unsigned)(key >> shift) & 255u], 1u);
        });
        __syncthreads();
        {
          // the bin holding the rank still to be located: scan the histogram from the top bin down, one
          // bin per thread (thread t owns bin 255 - t), instead of a serial walk by one thread
          const int rem = remaining_sh;
          const int mine = (int)hist[255 - tid];
          int tot_unused;
          const int above = block_exclusive_scan(mine, warp_tot, tot_unused);  // candidates in higher bins
          if (above < rem && above + mine >= rem) {  // exactly one thread
            prefix_sh = prefix | ((uint64_t)(255 - tid) << shift);
            remaining_sh = rem - above;
          }
        }
        __syncthreads();
      }
      thr = prefix_sh;
      need_eq = remaining_sh;  // 1 <= need_eq <= number of candidates equal to thr
      int eq = 0;
      for_each_key([&](uint64_t key) { eq += key == thr ? 1 : 0; });
      int tot;
      block_exclusive_scan(eq, warp_tot, tot);
      total_eq = tot;
    }
    // ordered compaction over positions
    int kept_base = 0, eq_base = 0;
    for (int j0 = 0; j0 < n; j0 += kSelThreads) {
      const int j = j0 + tid;
      int is_eq = 0, gt = 0;
      if (j < nc && kb > 0) {
        const uint64_t key = score_key(acc0[j], j, n, c.score_mode);
        is_eq = key == thr;
        gt = key > thr;
      }
      int tot_eq_chunk;
      const int eq_rank = eq_base + block_exclusive_scan(is_eq, warp_tot, tot_eq_chunk);
      // among equal scores the highest positions are the strongest: skip the first total_eq - need_eq
      const int keep = (j < n) && (j >= nc || gt || (is_eq && eq_rank >= total_eq - need_eq));
      int tot_keep;
      const int dst = kept_base + block_exclusive_scan(keep, warp_tot, tot_keep);
      if (keep && dst < B && H2O_IN_RANGE(dst, m, c.status)) kept[dst] = j;
      kept_base += tot_keep;
      eq_base += tot_eq_chunk;
    }
    if (tid == 0 && kept_base != B) atomicCAS(c.status, 0, H2O_ERR_STATE);
  }
  __syncthreads();

  // gather into the unit's slots
  const int64_t s0 = mt.slot_off;
  const int64_t stride = (int64_t)c.n_heads * D;
  const int64_t base = ((int64_t)lo * c.n_heads + h) * D;
  T* Kb = reinterpret_cast<T*>(c.K) + s0 * D;
  T* Vb = reinterpret_cast<T*>(c.V) + s0 * D;
  for (int x = tid; x < m; x += kSelThreads) {
    const int j = kept[x];
    if (!H2O_IN_RANGE(j, n, c.status) || !H2O_IN_RANGE(s0 + x, c.total_slots, c.status)) continue;
    c.acc[s0 + x] = acc0[j];
    c.pos[s0 + x] = j;
  }
  if (c.kv4 == 0)  // (4-bit slots are filled by their own gather kernel, from the positions written above)
#pragma unroll 4
  for (int x = tid; x < m * LPR; x += kSelThreads) {
    const int slot = x / LPR, ch = x % LPR;
    if (!H2O_IN_RANGE(kept[slot], n, c.status) || !H2O_IN_RANGE(s0 + slot, c.total_slots, c.status)) continue;
    const int64_t src = base + (int64_t)kept[slot] * stride + ch * VEC;
    *reinterpret_cast<uint4*>(Kb + (int64_t)slot * D + ch * VEC) = *reinterpret_cast<const uint4*>(k + src);
    *reinterpret_cast<uint4*>(Vb + (int64_t)slot * D + ch * VEC) = *reinterpret_cast<const uint4*>(v + src);
  }
  if (tid == 0) {
    c.count[su] = m;
    c.tpos[su] = n;
  }
}

template <typename T, int D, int KPT>
cudaError_t launch_kpt(const CacheView& c, const PrefillScratch& s, int max_B, const void* k, const void* v,
                       cudaStream_t stream) {
  const size_t smem = sizeof(int32_t) * (size_t)(max_B > 0 ? max_B : 1);
  if (smem > 48 * 1024) {
    cudaError_t e =
        cudaFuncSetAttribute(select_gather_kernel<T, D, KPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  select_gather_kernel<T, D, KPT><<<c.units, kSelThreads, smem, stream>>>(c, s, static_cast<const T*>(k),
                                                                         static_cast<const T*>(v));
  return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch(const CacheView& c, const PrefillScratch& s, int max_B, int max_seqlen, const void* k, const void* v,
                   cudaStream_t stream) {
  if (max_seqlen <= 2 * kSelThreads) return launch_kpt<T, D, 2>(c, s, max_B, k, v, stream);
  if (max_seqlen <= 8 * kSelThreads) return launch_kpt<T, D, 8>(c, s, max_B, k, v, stream);
  if (max_seqlen <= 16 * kSelThreads) return launch_kpt<T, D, 16>(c, s, max_B, k, v, stream);
  return launch_kpt<T, D, 0>(c, s, max_B, k, v, stream);
}

// F_score of every unit: the sum of h(accumulated score) over its occupied slots (the score function of
// the eviction policy's definition; h: 0 identity, 1 sqrt(z + 1), 2 log(z + 1), see the remark on h).
// Reporting only.  fp64, fixed summation order.
constexpr int kFsThreads = 128;
__global__ void __launch_bounds__(kFsThreads) fscore_kernel(CacheView c, int hkind, double* __restrict__ out) {
  __shared__ double part[kFsThreads];
  const UnitMeta mt = c.meta[blockIdx.x];
  const int cnt = c.count[blockIdx.x];
  const double* acc = c.acc + mt.slot_off;
  double f = 0.0;
  for (int x = threadIdx.x; x < cnt; x += kFsThreads) {
    const double a = acc[x];
    f += hkind == 1 ? sqrt(a + 1.0) : hkind == 2 ? log(a + 1.0) : a;
  }
  part[threadIdx.x] = f;
  __syncthreads();
  for (int w = kFsThreads / 2; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) part[threadIdx.x] += part[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[mt.unit] = part[0];
}

}  // namespace

cudaError_t launch_select_gather(const CacheView& c, const PrefillScratch& s, int dtype, int max_B, int max_seqlen,
                                 const void* k, const void* v, cudaStream_t stream) {
  if (dtype == H2O_F32) {
    if (c.head_dim == 64) return launch<float, 64>(c, s, max_B, max_seqlen, k, v, stream);
    return launch<float, 128>(c, s, max_B, max_seqlen, k, v, stream);
  }
  if (c.head_dim == 64) return launch<__nv_bfloat16, 64>(c, s, max_B, max_seqlen, k, v, stream);
  return launch<__nv_bfloat16, 128>(c, s, max_B, max_seqlen, k, v, stream);
}

}  // namespace h2o

namespace h2o {
cudaError_t launch_fscore(const CacheView& c, int hkind, double* out, cudaStream_t stream) {
  fscore_kernel<<<c.units, kFsThreads, 0, stream>>>(c, hkind, out);
  return cudaGetLastError();
}
}  // namespace h2o
