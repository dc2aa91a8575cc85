// Fused decode step for grouped-query attention: G query heads share the keys and values of one (sequence, head)
// unit.  One thread block per unit; every K row and every V row is read once for all G queries, which is the point
// of the sharing: the step moves the bytes of ONE head's cache for G heads' attention.
//
// The paper evicts per head and knows no such sharing (its comparison with a method that accumulates scores across
// heads is the nearest text).  Reading: every query head of the group attends the unit's entries with its own
// softmax; a key's accumulated score grows by the SUM of the probabilities the group's heads gave it (Algorithm 2's
// accumulation, once per query head); one victim per unit, chosen as always.
//
// Shape: a K pass (G dot products per loaded row, raw scores to shared memory), a softmax per query head (warp g
// does head g), a V pass (G weighted sums per loaded row), then the usual tail: fp64 accumulation, victim search by
// (score, position), in-place write of the new row.  Plain 16-byte loads, four rows in flight per half warp; this
// kernel is the plain variant of the step for every dtype and head size (no bulk-copy ring, no cluster split);
// bf16 / head_dim 128 caches whose staging fits take the streaming kernel of decode_two_pass.cu instead.
#include <climits>

#include "h2o_internal.cuh"
#include "step_common.cuh"

namespace h2o {

namespace {

using namespace step;

constexpr int kGqThreads = 256;
constexpr int kGqWarps = kGqThreads / 32;

template <typename T, int D, int G>
__global__ void __launch_bounds__(kGqThreads)
decode_gqa_kernel(CacheView c, const T* __restrict__ q, const T* __restrict__ k_new, const T* __restrict__ v_new,
                  T* __restrict__ out, int32_t* __restrict__ evicted_pos, int pitch) {
  constexpr int VEC = Vec16<T>::N, LPR = D / VEC, RPW = 32 / LPR, RPC = kGqWarps * RPW, UNROLL = 4;
  extern __shared__ __align__(16) unsigned char dyn[];
  float* s = reinterpret_cast<float*>(dyn);                  // [G][pitch]: raw scores, then probabilities
  float* red = s + G * pitch;                                // [warps][G][D]: per-warp partial outputs
  __shared__ float sm_m[G], sm_l[G];
  __shared__ Cand wbest[kGqWarps];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPR, ch = lane % LPR;
  const int su = blockIdx.x;  // launch position
  const UnitMeta mt = c.meta[su];
  // the previous kernel of the stream may have written this cache or produced q / k_new / v_new
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int u = mt.unit, r = mt.rwin, B = mt.kbud + mt.rwin;
  int cnt = c.count[su];
  if (!H2O_IN_RANGE(u, c.units, c.status) || !H2O_IN_RANGE(cnt, B + 1, c.status) ||
      !H2O_IN_RANGE(mt.slot_off + (cnt > 0 ? cnt - 1 : 0), c.total_slots, c.status))
    cnt = 0;
  const int t = c.tpos[su];
  const T* Kb = reinterpret_cast<const T*>(c.K) + mt.slot_off * D;
  const T* Vb = reinterpret_cast<const T*>(c.V) + mt.slot_off * D;
  const T* qu = q + (int64_t)u * G * D;  // the group's query heads are consecutive
  const T* ku = k_new + (int64_t)u * D;
  const T* vu = v_new + (int64_t)u * D;

  // ---- K pass: G scores per row --------------------------------------------------------------------
  float qf[G][VEC];
#pragma unroll
  for (int g = 0; g < G; ++g) Vec16<T>::load(qu + g * D + ch * VEC, qf[g]);
  for (int base = warp * RPW; base < cnt; base += RPC * UNROLL) {
    float kf[UNROLL][VEC];
#pragma unroll
    for (int un = 0; un < UNROLL; ++un) {
      const int row = base + un * RPC + sub;
      if (row < cnt) {
        Vec16<T>::load(Kb + (int64_t)row * D + ch * VEC, kf[un]);
      } else {
#pragma unroll
        for (int v = 0; v < VEC; ++v) kf[un][v] = 0.f;
      }
    }
#pragma unroll
    for (int un = 0; un < UNROLL; ++un) {
      const int row = base + un * RPC + sub;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float part = 0.f;
#pragma unroll
        for (int v = 0; v < VEC; ++v) part = fmaf(qf[g][v], kf[un][v], part);
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        if (ch == 0 && row < cnt) s[g * pitch + row] = c.scale * part;
      }
    }
  }
  if (warp == 0 && sub == 0) {  // the new token against itself, per query head
    float kf[VEC];
    Vec16<T>::load(ku + ch * VEC, kf);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float part = 0.f;
#pragma unroll
      for (int v = 0; v < VEC; ++v) part = fmaf(qf[g][v], kf[v], part);
#pragma unroll
      for (int off = LPR / 2; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu >> (32 - LPR), part, off);
      if (ch == 0) s[g * pitch + cnt] = c.scale * part;
    }
  }
  __syncthreads();

  // ---- softmax per query head: warp g does head g (G <= 8 warps) -------------------------------------
  const int total = cnt + 1;
  for (int g = warp; g < G; g += kGqWarps) {
    float* sg = s + g * pitch;
    float mx = -INFINITY;
    for (int x = lane; x < total; x += 32) mx = fmaxf(mx, sg[x]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int x = lane; x < total; x += 32) {
      const float e = expf(sg[x] - mx);
      sg[x] = e;
      sum += e;
    }
    sum = warp_sum(sum);
    const float inv = 1.0f / sum;
    for (int x = lane; x < total; x += 32) sg[x] *= inv;
    if (lane == 0) {
      sm_m[g] = mx;
      sm_l[g] = sum;
    }
  }
  __syncthreads();

  // ---- V pass: G weighted sums per row ---------------------------------------------------------------
  float o[G][VEC];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int v = 0; v < VEC; ++v) o[g][v] = 0.f;
  for (int base = warp * RPW; base < cnt; base += RPC * UNROLL) {
    float vf[UNROLL][VEC];
#pragma unroll
    for (int un = 0; un < UNROLL; ++un) {
      const int row = base + un * RPC + sub;
      if (row < cnt) {
        Vec16<T>::load(Vb + (int64_t)row * D + ch * VEC, vf[un]);
      } else {
#pragma unroll
        for (int v = 0; v < VEC; ++v) vf[un][v] = 0.f;
      }
    }
#pragma unroll
    for (int un = 0; un < UNROLL; ++un) {
      const int row = base + un * RPC + sub;
      if (row < cnt) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const float pr = s[g * pitch + row];
#pragma unroll
          for (int v = 0; v < VEC; ++v) o[g][v] = fmaf(pr, vf[un][v], o[g][v]);
        }
      }
    }
  }
  // the warp's row groups, then the warps (fixed order), then the new token's own value
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int v = 0; v < VEC; ++v)
#pragma unroll
      for (int off = LPR; off < 32; off <<= 1) o[g][v] += __shfl_xor_sync(0xffffffffu, o[g][v], off);
  if (sub == 0) {
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int v = 0; v < VEC; ++v) red[(warp * G + g) * D + ch * VEC + v] = o[g][v];
  }
  __syncthreads();
  for (int i = tid; i < G * D; i += kGqThreads) {
    const int g = i / D, x = i % D;
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < kGqWarps; ++w) acc += red[(w * G + g) * D + x];
    float vs;
    if constexpr (sizeof(T) == 4) vs = *reinterpret_cast<const float*>(vu + x);
    else vs = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vu + x));
    acc = fmaf(s[g * pitch + cnt], vs, acc);
    if constexpr (sizeof(T) == 4) reinterpret_cast<float*>(out)[((int64_t)u * G + g) * D + x] = acc;
    else reinterpret_cast<__nv_bfloat16*>(out)[((int64_t)u * G + g) * D + x] = __float2bfloat16_rn(acc);
  }

  // ---- accumulate (every head's probability), victim, in-place write ----------------------------------
  const bool full = cnt >= B;
  double* acc_g = c.acc + mt.slot_off;
  const int32_t* pos_g = c.pos + mt.slot_off;
  Cand best = cand_none();
  for (int x = tid; x < cnt; x += kGqThreads) {
    double px = 0.0;
#pragma unroll
    for (int g = 0; g < G; ++g) px += (double)s[g * pitch + x];
    const double a = acc_g[x] + px;
    acc_g[x] = a;
    const int ps = pos_g[x];
    if (full && ps <= t - r) {
      const double rank = c.score_mode == 1 ? a / (double)(t - ps + 1) : a;
      const Cand cx{(unsigned long long)__double_as_longlong(rank), ps, x};
      if (cand_before(cx, best)) best = cx;
    }
  }
  double p_self = 0.0;
#pragma unroll
  for (int g = 0; g < G; ++g) p_self += (double)s[g * pitch + cnt];
  if (tid == 0 && full && r == 0) {  // without a recent window the new token competes too
    const Cand cs{(unsigned long long)__double_as_longlong(p_self), t, -2};
    if (cand_before(cs, best)) best = cs;
  }
  best = warp_argmin(best);
  if (lane == 0) wbest[warp] = best;
  __syncthreads();
  if (warp == 0) {
    Cand b = lane < kGqWarps ? wbest[lane] : cand_none();
    b = warp_argmin(b);
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
    if (slot >= 0 && (!H2O_IN_RANGE(slot, B, c.status) || !H2O_IN_RANGE(mt.slot_off + slot, c.total_slots, c.status))) slot = -1;
    if (lane == 0) {
      if (!full) c.count[su] = cnt + 1;
      if (slot >= 0) {
        c.acc[mt.slot_off + slot] = p_self;
        c.pos[mt.slot_off + slot] = t;
      }
      if (evicted_pos) evicted_pos[u] = ev;
      c.tpos[su] = t + 1;
    }
    if (slot >= 0) {
      for (int i = lane; i < 2 * LPR; i += 32) {  // the new K/V row goes straight into the freed slot
        const T* src = (i < LPR ? ku : vu) + (i % LPR) * VEC;
        T* dst = reinterpret_cast<T*>(i < LPR ? c.K : c.V) + (mt.slot_off + slot) * D + (i % LPR) * VEC;
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
      }
    }
  }
}

template <typename T, int D, int G>
cudaError_t launch_g(const CacheView& c, int max_B, const void* q, const void* k_new, const void* v_new, void* out,
                     int32_t* evicted_pos, cudaStream_t stream) {
  const int pitch = (max_B + 1 + 3) & ~3;
  const size_t smem = (size_t)G * pitch * sizeof(float) + (size_t)kGqWarps * G * D * sizeof(float);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  static unsigned long long attr_flags = 0;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_gqa_kernel<T, D, G>), 200 * 1024, &attr_flags);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)c.units);
  cfg.blockDim = dim3(kGqThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_gqa_kernel<T, D, G>, c, static_cast<const T*>(q), static_cast<const T*>(k_new),
                            static_cast<const T*>(v_new), static_cast<T*>(out), evicted_pos, pitch);
}

template <typename T, int D>
cudaError_t launch_td(const CacheView& c, int max_B, const void* q, const void* k_new, const void* v_new, void* out,
                      int32_t* evicted_pos, cudaStream_t stream) {
  switch (c.group) {
    case 2: return launch_g<T, D, 2>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
    case 4: return launch_g<T, D, 4>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
    case 8: return launch_g<T, D, 8>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

size_t decode_gqa_smem_bytes(int group, int max_B, int head_dim) {
  const int pitch = (max_B + 1 + 3) & ~3;
  return (size_t)group * pitch * sizeof(float) + (size_t)kGqWarps * group * head_dim * sizeof(float);
}

cudaError_t launch_decode_gqa(const CacheView& c, int dtype, int max_B, bool cache_is_quiescent, bool all_full, const void* q,
                              const void* k_new, const void* v_new, void* out, int32_t* evicted_pos, cudaStream_t stream) {
  if (decode_two_pass_supported(dtype, c.head_dim, c.group, max_B))
    return launch_decode_two_pass(c, 1, (max_B + 3) & ~3, cache_is_quiescent, all_full, q, k_new, v_new, out, evicted_pos, stream);
  if (dtype == H2O_F32) {
    if (c.head_dim == 64) return launch_td<float, 64>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
    return launch_td<float, 128>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
  }
  if (c.head_dim == 64) return launch_td<__nv_bfloat16, 64>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
  return launch_td<__nv_bfloat16, 128>(c, max_B, q, k_new, v_new, out, evicted_pos, stream);
}

}  // namespace h2o
