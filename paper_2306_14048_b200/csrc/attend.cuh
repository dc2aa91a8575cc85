// One query against `cnt` stored key/value rows (plus, optionally, the query's own
// token): scores, softmax, weighted sum of values — by one thread block.
//
// This is the ALU formulation (fp32 FMA on 16-byte vector loads).  The work is a
// matrix-vector product per unit, about one flop per byte read, so it is bound by
// memory traffic and is kept off the tensor cores on purpose.
//
// Thread mapping: a row of D elements is covered by LPR = D / VEC consecutive
// lanes, each holding one 16-byte chunk; a warp therefore handles RPW = 32 / LPR
// rows per pass and the block WARPS * RPW rows.  All reductions use a fixed order
// (xor butterflies, then warps in index order), so results are reproducible.
#pragma once

#include "h2o_internal.cuh"

namespace h2o {

template <typename T, int D, int THREADS>
struct Attend {
  static constexpr int VEC = Vec16<T>::N;
  static constexpr int LPR = D / VEC;
  static constexpr int RPW = 32 / LPR;
  static constexpr int WARPS = THREADS / 32;
  static constexpr int RPC = WARPS * RPW;
  static constexpr int UNROLL = 4;
  static_assert(D % VEC == 0 && LPR <= 32 && 32 % LPR == 0, "unsupported head_dim");

  struct Smem {
    float red[WARPS][D];  // per-warp partial outputs
    float scal[WARPS];    // scalar reductions
    float bcast[2];
  };

  __device__ __forceinline__ static float block_max(float x, Smem& sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    x = warp_max(x);
    __syncthreads();
    if (lane == 0) sm.scal[warp] = x;
    __syncthreads();
    float r = sm.scal[0];
#pragma unroll
    for (int w = 1; w < WARPS; ++w) r = fmaxf(r, sm.scal[w]);
    return r;
  }
  __device__ __forceinline__ static float block_sum(float x, Smem& sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    x = warp_sum(x);
    __syncthreads();
    if (lane == 0) sm.scal[warp] = x;
    __syncthreads();
    float r = sm.scal[0];
#pragma unroll
    for (int w = 1; w < WARPS; ++w) r += sm.scal[w];
    return r;
  }

  // On return p[0 .. cnt + has_self) holds the softmax probabilities (the query's own
  // token last), m / l the row maximum and the sum of exp(s - m), and the threads with
  // threadIdx.x < LPR hold, in o[], chunk threadIdx.x of the output row.
  // Row x holds the key of position x; with a sparse pattern (mask_kind != 0) the query, at position t_query
  // with recent window r_win, leaves out the rows key_attended() rejects (probability 0).
  __device__ static void run(const T* __restrict__ q, const T* __restrict__ Kb, const T* __restrict__ Vb,
                             int64_t row_stride, int cnt, const T* __restrict__ k_self,
                             const T* __restrict__ v_self, float c, float* __restrict__ p, Smem& sm,
                             float (&o)[VEC], float& m_out, float& l_out, int mask_kind = 0, int mask_a = 1,
                             int mask_b = 0, int t_query = 0, int r_win = 0) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane / LPR, ch = lane % LPR;
    const bool has_self = k_self != nullptr;
    const int total = cnt + (has_self ? 1 : 0);

    float qf[VEC];
    Vec16<T>::load(q + ch * VEC, qf);

    // ---- scores -----------------------------------------------------------
    for (int base = warp * RPW; base < cnt; base += RPC * UNROLL) {
      float kf[UNROLL][VEC];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int row = base + u * RPC + sub;
        if (row < cnt) {
          Vec16<T>::load(Kb + (int64_t)row * row_stride + ch * VEC, kf[u]);
        } else {
#pragma unroll
          for (int v = 0; v < VEC; ++v) kf[u][v] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int row = base + u * RPC + sub;
        float part = 0.f;
#pragma unroll
        for (int v = 0; v < VEC; ++v) part = fmaf(qf[v], kf[u][v], part);
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        if (ch == 0 && row < cnt)
          p[row] = key_attended(mask_kind, mask_a, mask_b, row, t_query, r_win) ? c * part : -INFINITY;
      }
    }
    if (has_self && warp == 0) {
      float part = 0.f;
      if (sub == 0) {
        float kf[VEC];
        Vec16<T>::load(k_self + ch * VEC, kf);
#pragma unroll
        for (int v = 0; v < VEC; ++v) part = fmaf(qf[v], kf[v], part);
      }
#pragma unroll
      for (int off = LPR / 2; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
      if (lane == 0) p[cnt] = c * part;
    }
    __syncthreads();

    // ---- softmax ----------------------------------------------------------
    float mx = -INFINITY;
    for (int x = tid; x < total; x += THREADS) mx = fmaxf(mx, p[x]);
    const float m = block_max(mx, sm);
    float sum = 0.f;
    for (int x = tid; x < total; x += THREADS) {
      const float e = expf(p[x] - m);
      p[x] = e;
      sum += e;
    }
    const float l = block_sum(sum, sm);
    for (int x = tid; x < total; x += THREADS) p[x] = p[x] / l;
    __syncthreads();
    m_out = m;
    l_out = l;

    // ---- weighted sum of values -------------------------------------------
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    for (int base = warp * RPW; base < cnt; base += RPC * UNROLL) {
      float vf[UNROLL][VEC];
      float pr[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int row = base + u * RPC + sub;
        if (row < cnt) {
          Vec16<T>::load(Vb + (int64_t)row * row_stride + ch * VEC, vf[u]);
          pr[u] = p[row];
        } else {
#pragma unroll
          for (int v = 0; v < VEC; ++v) vf[u][v] = 0.f;
          pr[u] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u)
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] = fmaf(pr[u], vf[u][v], acc[v]);
    }
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
      for (int v = 0; v < VEC; ++v) acc[v] += __shfl_xor_sync(0xffffffffu, acc[v], off);
    if (sub == 0) {
#pragma unroll
      for (int v = 0; v < VEC; ++v) sm.red[warp][ch * VEC + v] = acc[v];
    }
    __syncthreads();
    if (tid < LPR) {
#pragma unroll
      for (int v = 0; v < VEC; ++v) {
        float r = sm.red[0][tid * VEC + v];
#pragma unroll
        for (int w = 1; w < WARPS; ++w) r += sm.red[w][tid * VEC + v];
        o[v] = r;
      }
      if (has_self) {
        float vf[VEC];
        Vec16<T>::load(v_self + tid * VEC, vf);
        const float ps = p[cnt];
#pragma unroll
        for (int v = 0; v < VEC; ++v) o[v] = fmaf(ps, vf[v], o[v]);
      }
    }
  }
};

}  // namespace h2o
