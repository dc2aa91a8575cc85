// Pieces shared by the decode-step kernels (decode_two_pass.cu, decode_kv4.cu, decode_gqa.cu): the eviction
// candidate and its warp-wide minimum, the bounded wait on an mbarrier, the untiled bulk copy into shared memory.
#pragma once
#include <climits>
#include <cstdint>

#include "sm100_ptx.cuh"

namespace h2o {
namespace step {

// Eviction candidate (Algorithm 2 evicts the entry whose removal keeps the largest total score: with the summed
// score, the candidate with the smallest accumulated score; equal scores: the older position).  Accumulated scores
// are sums of probabilities (>= 0), so the bit pattern of the double orders like its value; comparing the integer
// key keeps the fp64 pipe out of the search.
struct Cand {
  unsigned long long key;  // bit pattern of the (non-negative) ranking score
  int pos, slot;           // slot -1: none, -2: the new token itself
};
__device__ __forceinline__ Cand cand_none() { return Cand{~0ull, INT_MAX, -1}; }
__device__ __forceinline__ bool cand_before(const Cand& a, const Cand& b) {
  if (a.slot == -1) return false;
  if (b.slot == -1) return true;
  return a.key < b.key || (a.key == b.key && a.pos < b.pos);
}
// Warp-wide minimum under that order; every lane gets the winner.  Three 32-bit hardware reductions (high word,
// low word, position) instead of five rounds of shuffled compares.
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
  Cand b;
  b.key = ((unsigned long long)mh << 32) | ml;
  b.pos = (int)mp;
  b.slot = __shfl_sync(0xffffffffu, a.slot, __ffs(who) - 1);
  return b;
}

// Bounded wait: false after kSpin unsuccessful polls (the caller records H2O_ERR_TIMEOUT and carries on).
constexpr uint32_t kSpin = 1u << 22;
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpin; ++it)
    if (ptx::mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> shared bulk copy (16-byte aligned addresses, size a multiple of 16), completion counted on `bar`
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   ptx::smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(ptx::smem_u32(bar))
               : "memory");
}

}  // namespace step
}  // namespace h2o
