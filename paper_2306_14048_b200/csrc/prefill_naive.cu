// Prompt attention and column sums on the fp32 FMA pipe, for every dtype and head_dim.
// This is the path of fp32 inputs (tensor cores would round them to TF32, which the
// exact-decision requirement cannot afford) and of head_dim 64.
//
//   rows kernel   : one thread block per (unit, query row i): P[i][0..i], out_i, m_i, l_i
//   colsum kernel : one thread per key column j: acc0[j] = sum_{i >= j} exp(c q_i.k_j - m_i) / l_i
//
// Paper: causal attention of the prompt (Appendix A pseudocode, prefill branch) and the
// accumulated score of Algorithm 2 evaluated for all prompt rows at once.
#include "attend.cuh"

namespace h2o {

namespace {

constexpr int kRowThreads = 128;
constexpr int kColThreads = 128;

template <typename T, int D>
__global__ void __launch_bounds__(kRowThreads)
prefill_rows_kernel(CacheView c, PrefillScratch s, const T* __restrict__ q, const T* __restrict__ k,
                    const T* __restrict__ v, T* __restrict__ out) {
  using A = Attend<T, D, kRowThreads>;
  constexpr int VEC = A::VEC, LPR = A::LPR;
  extern __shared__ float p[];
  __shared__ typename A::Smem sm;
  // blockIdx.y = (sequence, QUERY head); with grouped-query attention the query heads hq = h * G + g of a group
  // read the keys and values of head h
  const int G = c.group, HQ = c.n_heads * G;
  const int uq = blockIdx.y;
  const int seq = uq / HQ, hq = uq % HQ, h = hq / G;
  const int lo = s.cu[seq], n = s.cu[seq + 1] - lo;
  const int i = blockIdx.x;
  if (i >= n) return;
  if (!H2O_IN_RANGE(seq * c.n_heads + h, c.units, c.status) || !H2O_IN_RANGE((int64_t)lo + i, s.total_tokens, c.status)) return;
  const int64_t stride = (int64_t)c.n_heads * D, stride_q = (int64_t)HQ * D;
  const int64_t base = ((int64_t)lo * c.n_heads + h) * D, base_q = ((int64_t)lo * HQ + hq) * D;
  float o[VEC], m, l;
  const int r = c.mask_kind ? c.seq_rwin[seq] : 0;
  A::run(q + base_q + i * stride_q, k + base, v + base, stride, i + 1, nullptr, nullptr, c.scale, p, sm, o, m, l, c.mask_kind,
         c.mask_a, c.mask_b, i, r);
  if (threadIdx.x < LPR) Vec16<T>::store(out + base_q + i * stride_q + threadIdx.x * VEC, o);
  if (threadIdx.x == 0) {
    s.rowmax[(int64_t)hq * s.total_tokens + lo + i] = m;
    s.rowsum[(int64_t)hq * s.total_tokens + lo + i] = l;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kColThreads)
prefill_colsum_kernel(CacheView c, PrefillScratch s, const T* __restrict__ q, const T* __restrict__ k) {
  constexpr int VEC = Vec16<T>::N;
  const int u = blockIdx.y;
  const int seq = u / c.n_heads, h = u % c.n_heads;
  const int lo = s.cu[seq], n = s.cu[seq + 1] - lo;
  const int j0 = blockIdx.x * kColThreads;
  if (j0 >= n) return;
  const int j = j0 + threadIdx.x;
  const int G = c.group, HQ = c.n_heads * G;
  const int64_t stride = (int64_t)c.n_heads * D, stride_q = (int64_t)HQ * D;
  const int64_t base = ((int64_t)lo * c.n_heads + h) * D;

  float kf[D];
  if (j < n) {
#pragma unroll
    for (int x = 0; x < D; x += VEC) {
      float t[VEC];
      Vec16<T>::load(k + base + j * stride + x, t);
#pragma unroll
      for (int e = 0; e < VEC; ++e) kf[x + e] = t[e];
    }
  } else {
#pragma unroll
    for (int x = 0; x < D; ++x) kf[x] = 0.f;
  }
  const int r = c.mask_kind ? c.seq_rwin[seq] : 0;
  double a = 0.0;
  for (int g = 0; g < G; ++g) {  // the group's query heads one after the other: their column sums add up
    const int hq = h * G + g;
    const float* rowmax = s.rowmax + (int64_t)hq * s.total_tokens + lo;
    const float* rowsum = s.rowsum + (int64_t)hq * s.total_tokens + lo;
    for (int i = j0; i < n; ++i) {  // every thread of the block reads the same query row (broadcast)
      const T* qi = q + ((int64_t)lo * HQ + hq) * D + i * stride_q;
      float dot = 0.f;
#pragma unroll
      for (int x = 0; x < D; x += VEC) {
        float t[VEC];
        Vec16<T>::load(qi + x, t);
#pragma unroll
        for (int e = 0; e < VEC; ++e) dot = fmaf(t[e], kf[x + e], dot);
      }
      if (i >= j && key_attended(c.mask_kind, c.mask_a, c.mask_b, j, i, r))
        a += (double)(expf(c.scale * dot - rowmax[i]) / rowsum[i]);
    }
  }
  if (j < n && H2O_IN_RANGE((int64_t)lo + j, s.total_tokens, c.status)) s.acc0[(int64_t)h * s.total_tokens + lo + j] = a;
}

template <typename T, int D>
cudaError_t launch(const CacheView& c, const PrefillScratch& s, int max_seqlen, const void* q, const void* k,
                   const void* v, void* out, bool rows, bool colsum, cudaStream_t stream) {
  if (rows) {
    const size_t smem = sizeof(float) * (size_t)(max_seqlen + 1);
    if (smem > 48 * 1024) {
      cudaError_t e =
          cudaFuncSetAttribute(prefill_rows_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    dim3 grid_rows((unsigned)max_seqlen, (unsigned)(c.units * c.group));  // one block per query row of every query head
    prefill_rows_kernel<T, D><<<grid_rows, kRowThreads, smem, stream>>>(
        c, s, static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<T*>(out));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (colsum) {
    dim3 grid_cols((unsigned)((max_seqlen + kColThreads - 1) / kColThreads), (unsigned)c.units);
    prefill_colsum_kernel<T, D><<<grid_cols, kColThreads, 0, stream>>>(c, s, static_cast<const T*>(q),
                                                                      static_cast<const T*>(k));
    return cudaGetLastError();
  }
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_prefill_naive(const CacheView& c, const PrefillScratch& s, int dtype, int max_seqlen, const void* q,
                                 const void* k, const void* v, void* out, bool rows, bool colsum, cudaStream_t stream) {
  if (dtype == H2O_F32) {
    if (c.head_dim == 64) return launch<float, 64>(c, s, max_seqlen, q, k, v, out, rows, colsum, stream);
    return launch<float, 128>(c, s, max_seqlen, q, k, v, out, rows, colsum, stream);
  }
  if (c.head_dim == 64) return launch<__nv_bfloat16, 64>(c, s, max_seqlen, q, k, v, out, rows, colsum, stream);
  return launch<__nv_bfloat16, 128>(c, s, max_seqlen, q, k, v, out, rows, colsum, stream);
}

}  // namespace h2o
