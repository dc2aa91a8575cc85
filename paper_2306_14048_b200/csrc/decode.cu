// Fused decode step: scores over the occupied slots, softmax, weighted values,
// score accumulation, victim search and in-place replacement — one kernel, one
// thread block per (sequence, head), the cache read exactly once.
//
// Paper: Algorithm 2 loop body (scores, accumulate, argmax of F_score(G \ {v}) which
// for the summation score is the candidate with the smallest accumulated score) on
// the pre-allocated, overwritten-in-place cache of Section 4.2 / Appendix A.
#include <cfloat>

#include "attend.cuh"

namespace h2o {

namespace {

constexpr int kDecodeThreads = 256;

struct Cand {
  double acc;
  int pos;
  int slot;  // -1: none, -2: the new token itself
};

__device__ __forceinline__ bool cand_before(const Cand& a, const Cand& b) {
  if (a.slot == -1) return false;
  if (b.slot == -1) return true;
  return a.acc < b.acc || (a.acc == b.acc && a.pos < b.pos);
}

__device__ __forceinline__ Cand cand_shfl_xor(const Cand& a, int off) {
  Cand b;
  b.acc = __shfl_xor_sync(0xffffffffu, a.acc, off);
  b.pos = __shfl_xor_sync(0xffffffffu, a.pos, off);
  b.slot = __shfl_xor_sync(0xffffffffu, a.slot, off);
  return b;
}

template <typename T, int D>
__global__ void __launch_bounds__(kDecodeThreads)
decode_kernel(CacheView c, const T* __restrict__ q, const T* __restrict__ k_new, const T* __restrict__ v_new,
              T* __restrict__ out, int32_t* __restrict__ evicted_pos) {
  using A = Attend<T, D, kDecodeThreads>;
  constexpr int VEC = A::VEC, LPR = A::LPR, WARPS = A::WARPS;
  extern __shared__ float p[];  // [cnt + 1] scores, then probabilities
  __shared__ typename A::Smem sm;
  __shared__ Cand wbest[WARPS];
  __shared__ int victim_sh;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = c.order[blockIdx.x];
  const int cnt = c.count[u];
  const int t = c.tpos[u];
  const int r = c.rwin[u];
  const int B = c.kbud[u] + r;
  const int64_t s0 = c.slot_off[u];
  T* Kb = reinterpret_cast<T*>(c.K) + s0 * D;
  T* Vb = reinterpret_cast<T*>(c.V) + s0 * D;
  double* acc = c.acc + s0;
  int32_t* pos = c.pos + s0;
  const T* qu = q + (int64_t)u * D;
  const T* ku = k_new + (int64_t)u * D;
  const T* vu = v_new + (int64_t)u * D;

  float o[VEC], m, l;
  A::run(qu, Kb, Vb, D, cnt, ku, vu, c.scale, p, sm, o, m, l);
  if (tid < LPR) Vec16<T>::store(out + (int64_t)u * D + tid * VEC, o);

  // accumulate (Algorithm 2: o~_i = o~_{i-1} + o_i) and search the victim among the
  // entries outside the recent window
  const bool full = cnt >= B;
  Cand best{DBL_MAX, INT_MAX, -1};
  for (int x = tid; x < cnt; x += kDecodeThreads) {
    const double a = acc[x] + (double)p[x];
    acc[x] = a;
    const int px = pos[x];
    if (full && px <= t - r) {
      const Cand cx{a, px, x};
      if (cand_before(cx, best)) best = cx;
    }
  }
  if (full && r == 0 && tid == 0) {  // without a recent window the new token competes too
    const Cand cs{(double)p[cnt], t, -2};
    if (cand_before(cs, best)) best = cs;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const Cand other = cand_shfl_xor(best, off);
    if (cand_before(other, best)) best = other;
  }
  if (lane == 0) wbest[warp] = best;
  __syncthreads();
  if (tid == 0) {
    Cand b = wbest[0];
#pragma unroll
    for (int w = 1; w < WARPS; ++w)
      if (cand_before(wbest[w], b)) b = wbest[w];
    int slot, ev;
    if (!full) {
      slot = cnt;
      ev = -1;
      c.count[u] = cnt + 1;
    } else if (b.slot == -2) {
      slot = -1;
      ev = t;
    } else if (b.slot >= 0) {
      slot = b.slot;
      ev = b.pos;
    } else {  // a full cache always has a candidate; record instead of corrupting
      slot = -1;
      ev = -1;
      atomicCAS(c.status, 0, H2O_ERR_STATE);
    }
    if (slot >= 0) {
      acc[slot] = (double)p[cnt];
      pos[slot] = t;
    }
    if (evicted_pos) evicted_pos[u] = ev;
    c.tpos[u] = t + 1;
    victim_sh = slot;
  }
  __syncthreads();
  const int slot = victim_sh;
  if (slot >= 0 && tid < 2 * LPR) {  // in-place replacement: the new K/V row goes into the freed slot
    const int ch = tid % LPR;
    const uint4 val = *reinterpret_cast<const uint4*>((tid < LPR ? ku : vu) + ch * VEC);
    *reinterpret_cast<uint4*>((tid < LPR ? Kb : Vb) + (int64_t)slot * D + ch * VEC) = val;
  }
}

template <typename T, int D>
cudaError_t launch(const CacheView& c, int max_B, const void* q, const void* k_new, const void* v_new, void* out,
                   int32_t* evicted_pos, cudaStream_t stream) {
  const size_t smem = sizeof(float) * (size_t)(max_B + 1);
  decode_kernel<T, D><<<c.units, kDecodeThreads, smem, stream>>>(
      c, static_cast<const T*>(q), static_cast<const T*>(k_new), static_cast<const T*>(v_new), static_cast<T*>(out),
      evicted_pos);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode(const CacheView& c, int dtype, int max_B, const void* q, const void* k_new, const void* v_new,
                          void* out, int32_t* evicted_pos, cudaStream_t stream) {
  if (dtype == H2O_F32) {
    if (c.head_dim == 64) return launch<float, 64>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
    return launch<float, 128>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
  }
  if (c.head_dim == 64) return launch<__nv_bfloat16, 64>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
  return launch<__nv_bfloat16, 128>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
}

}  // namespace h2o
