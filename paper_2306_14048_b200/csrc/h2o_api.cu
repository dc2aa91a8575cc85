// Host side of the C ABI declared in include/h2o.h: argument checks, workspace
// carving, call-order state machine and kernel launches.  No device memory is
// allocated here; everything lives in the caller's workspace / scratch.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <numeric>
#include <vector>

#include "h2o_internal.cuh"

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxSlotsPerUnit = 65536;  // bounded by the decode kernel's shared-memory score rows
constexpr int kMaxSlotsPerUnitKv4 = 8192;  // 4-bit slots: one thread block per unit, its scores and staging in shared memory
constexpr int kMaxPromptLen = 49151;     // the ALU prefill keeps one score row in shared memory
constexpr int kMaxChunk = 8192;          // slots per decode thread block
constexpr int kMaxUnits = 65535;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

size_t elem_size(int dtype) { return dtype == H2O_F32 ? 4 : 2; }  // of q / k / v / out
// dtype of the inputs as the kernels' template selectors know it
int input_dtype(int dtype) { return dtype == H2O_BF16_KV4 ? H2O_BF16 : dtype; }
size_t slot_row_bytes(const h2o_config_t* cfg) {
  return cfg->dtype == H2O_BF16_KV4 ? h2o::kv4_row_bytes() : (size_t)cfg->head_dim * elem_size(cfg->dtype);
}

struct Layout {
  size_t K, V, acc, pos, count, tpos, status, meta, seq_rwin, total;
  int64_t total_slots;
  int max_B;
};

// 0 = fine, otherwise an H2O_ERR_* code.
int check_config(const h2o_config_t* cfg) {
  if (!cfg || !cfg->heavy_budget || !cfg->recent_window) return H2O_ERR_INVALID_ARG;
  if (cfg->batch < 1 || cfg->n_heads < 1 || cfg->device < 0) return H2O_ERR_INVALID_ARG;
  if (cfg->dtype != H2O_F32 && cfg->dtype != H2O_BF16 && cfg->dtype != H2O_BF16_KV4) return H2O_ERR_UNSUPPORTED;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return H2O_ERR_UNSUPPORTED;
  if (cfg->dtype == H2O_BF16_KV4 && cfg->head_dim != 128) return H2O_ERR_UNSUPPORTED;
  if ((int64_t)cfg->batch * cfg->n_heads > kMaxUnits) return H2O_ERR_UNSUPPORTED;
  for (int s = 0; s < cfg->batch; ++s) {
    const int64_t k = cfg->heavy_budget[s], r = cfg->recent_window[s];
    if (k < 0 || r < 0 || k + r < 1) return H2O_ERR_INVALID_ARG;
    if (k + r > kMaxSlotsPerUnit) return H2O_ERR_UNSUPPORTED;
    if (cfg->dtype == H2O_BF16_KV4 && k + r > kMaxSlotsPerUnitKv4) return H2O_ERR_UNSUPPORTED;
  }
  if (std::isnan(cfg->softmax_scale) || std::isinf(cfg->softmax_scale)) return H2O_ERR_INVALID_ARG;
  const int G = cfg->query_group;
  if (G < 0) return H2O_ERR_INVALID_ARG;
  if (G > 1) {  // grouped-query attention
    if (G != 2 && G != 4 && G != 8) return H2O_ERR_UNSUPPORTED;
    if (cfg->dtype == H2O_BF16_KV4) return H2O_ERR_UNSUPPORTED;
    for (int s = 0; s < cfg->batch; ++s)  // the group's scores of one unit stay in shared memory
      if (h2o::decode_gqa_smem_bytes(G, cfg->heavy_budget[s] + cfg->recent_window[s], cfg->head_dim) > 200 * 1024)
        return H2O_ERR_UNSUPPORTED;
  }
  return H2O_OK;
}
int group_of(const h2o_config_t* cfg) { return cfg->query_group > 1 ? cfg->query_group : 1; }

Layout make_layout(const h2o_config_t* cfg) {
  Layout L{};
  int64_t slots = 0;
  int max_B = 0;
  for (int s = 0; s < cfg->batch; ++s) {
    const int B = cfg->heavy_budget[s] + cfg->recent_window[s];
    slots += (int64_t)((B + 3) & ~3) * cfg->n_heads;  // units start on a multiple of 4 slots (16-byte bulk copies)
    max_B = std::max(max_B, B);
  }
  const size_t units = (size_t)cfg->batch * cfg->n_heads;
  const size_t row = slot_row_bytes(cfg);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes);
    return at;
  };
  L.K = take((size_t)slots * row);
  L.V = take((size_t)slots * row);
  L.acc = take((size_t)slots * sizeof(double));
  L.pos = take((size_t)slots * sizeof(int32_t));
  L.count = take(units * sizeof(int32_t));
  L.tpos = take(units * sizeof(int32_t));
  L.status = take(sizeof(int32_t));
  L.meta = take(units * sizeof(h2o::UnitMeta));
  L.seq_rwin = take((size_t)cfg->batch * sizeof(int32_t));
  L.total = off;
  L.total_slots = slots;
  L.max_B = max_B;
  return L;
}

struct ScratchLayout {
  size_t rowstat, acc0, cu, total;
};

ScratchLayout make_scratch_layout(const h2o_config_t* cfg, int64_t total_tokens) {
  ScratchLayout S{};
  const size_t cells = (size_t)total_tokens * cfg->n_heads;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes);
    return at;
  };
  S.rowstat = take(cells * group_of(cfg) * 2 * sizeof(float));  // row maximum and row sum per QUERY head (planar or interleaved)
  S.acc0 = take(cells * sizeof(double));
  // cu_seqlens, two work counters, first item index of every group of units (at most one group per unit)
  S.cu = take(((size_t)cfg->batch + 1 + 2 + (size_t)cfg->batch * cfg->n_heads * group_of(cfg) + 1) * sizeof(int32_t));
  S.total = off;
  return S;
}

// Failed: a launch of a multi-kernel call was refused after earlier work of the same call had been enqueued; the
// workspace is then partly written and only h2o_cache_reset (or destroy) is accepted.
enum class Phase { Empty, Prefilled, Decoding, Failed };

}  // namespace

struct h2o_cache {
  h2o_config_t cfg;
  std::vector<int32_t> heavy, recent, cu;
  std::vector<h2o::UnitMeta> meta;  // launch order
  int split, chunk, stages;
  int prefill_path;  // 0 = automatic, 1 = force the ALU kernels
  int chunk_path;    // 0 = automatic, 1 = force one decode-step kernel per token in h2o_decode_chunk
  int decode_path;   // 0 = automatic, 1 = the online-softmax step kernel, 2 = the two-pass streaming kernel
  double mean_budget;  // mean of k + r over the sequences
  // tokens every unit of sequence s has been given (prompt + decode steps); < 0: unknown (attached cache)
  std::vector<int64_t> seen;
  Layout layout;
  h2o::CacheView view;
  Phase phase;
  cudaEvent_t prefill_events[4] = {nullptr, nullptr, nullptr, nullptr};  // see h2o_debug_set_prefill_events
};

namespace {

// Which cache did this library's most recent launch on a stream write?  Only this library writes a
// cache workspace, so if the answer is "another cache" (or the stream has since run foreign work,
// which completes our earlier kernel first), a decode kernel may read its cache before the preceding
// kernel of the stream has finished.  Unknown streams are treated as "this cache" (no early reads).
class LastWriter {
 public:
  // returns true if the last recorded writer on `stream` is a different cache; then records `cache`
  bool note_and_check(cudaStream_t stream, const void* cache) {
    std::lock_guard<std::mutex> lock(mu_);
    for (auto& e : entries_) {
      if (e.stream == stream) {
        const bool other = e.cache != nullptr && e.cache != cache;
        e.cache = cache;
        return other;
      }
    }
    if (entries_.size() >= 64) entries_.erase(entries_.begin());
    entries_.push_back({stream, cache});
    return false;
  }
  void forget(const void* cache) {
    std::lock_guard<std::mutex> lock(mu_);
    for (auto& e : entries_)
      if (e.cache == cache) e.cache = nullptr;
  }

 private:
  struct Entry {
    cudaStream_t stream;
    const void* cache;
  };
  std::mutex mu_;
  std::vector<Entry> entries_;
};
LastWriter g_last_writer;
bool g_early_prefetch = true;  // diagnostic switch, see h2o_debug_set_early_prefetch

// Device-side address of a host buffer the GPU can access directly (pinned or registered, 16-byte
// aligned); nullptr for pageable or foreign memory.
void* device_alias(const void* host_ptr) {
  cudaPointerAttributes attr{};
  if (cudaPointerGetAttributes(&attr, host_ptr) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  if (attr.type != cudaMemoryTypeHost || !attr.devicePointer) return nullptr;
  if (reinterpret_cast<uintptr_t>(attr.devicePointer) % 16 != 0) return nullptr;
  return attr.devicePointer;
}

// Does the host know that every unit holds exactly its budget of entries?
bool all_units_full(const h2o_cache* c) {
  for (int s = 0; s < c->cfg.batch; ++s)
    if (c->seen[s] < (int64_t)c->heavy[s] + c->recent[s]) return false;  // also when unknown (-1)
  return true;
}
void advance_seen(h2o_cache* c, int64_t tokens) {
  for (auto& x : c->seen)
    if (x >= 0) x += tokens;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = prev == dev || cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (ok && prev >= 0) {
      int cur = -1;
      if (cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
  }
};

}  // namespace

namespace h2o {
const h2o_config_t* cache_config(const h2o_cache_t* cache) { return &cache->cfg; }
}  // namespace h2o

extern "C" {

size_t h2o_cache_workspace_bytes(const h2o_config_t* cfg) {
  if (check_config(cfg) != H2O_OK) return 0;
  return make_layout(cfg).total;
}

size_t h2o_prefill_scratch_bytes(const h2o_config_t* cfg, int64_t total_tokens) {
  if (check_config(cfg) != H2O_OK || total_tokens < 1 || total_tokens > INT32_MAX) return 0;
  return make_scratch_layout(cfg, total_tokens).total;
}

static int create_impl(h2o_cache_t** out, const h2o_config_t* cfg, void* dev_workspace, size_t workspace_bytes,
                       bool attach) {
  if (!out) return H2O_ERR_INVALID_ARG;
  const int rc = check_config(cfg);
  if (rc != H2O_OK) return rc;
  if (!dev_workspace) return H2O_ERR_INVALID_ARG;
  const Layout L = make_layout(cfg);
  if (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(dev_workspace) % kAlign) != 0) return H2O_ERR_WORKSPACE;

  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  if (cfg->device >= ndev) return H2O_ERR_INVALID_ARG;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, cfg->device) != cudaSuccess) return H2O_ERR_CUDA;
  if (major != 10) return H2O_ERR_UNSUPPORTED;  // the kernels are built for sm_100a only
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return H2O_ERR_CUDA;

  h2o_cache* c = new (std::nothrow) h2o_cache();
  if (!c) return H2O_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->heavy.assign(cfg->heavy_budget, cfg->heavy_budget + cfg->batch);
  c->recent.assign(cfg->recent_window, cfg->recent_window + cfg->batch);
  c->cfg.heavy_budget = c->heavy.data();
  c->cfg.recent_window = c->recent.data();
  c->layout = L;
  c->phase = Phase::Empty;

  const int units = cfg->batch * cfg->n_heads;
  std::vector<h2o::UnitMeta> meta(units);
  int64_t at = 0;
  for (int u = 0; u < units; ++u) {
    const int s = u / cfg->n_heads;
    meta[u] = h2o::UnitMeta{at, u, c->heavy[s], c->recent[s], 0};
    at += (c->heavy[s] + c->recent[s] + 3) & ~3;
  }
  std::stable_sort(meta.begin(), meta.end(), [](const h2o::UnitMeta& a, const h2o::UnitMeta& b) {
    return a.kbud + a.rwin > b.kbud + b.rwin;  // longest first
  });
  c->meta = meta;
  // Thread blocks per unit.  One block per unit unless there are fewer units than SMs: sharing a
  // unit costs three cluster barriers per step, which only pays when SMs would otherwise idle.
  int split = 1;
  const int sms = h2o::sm_count();
  while (split < 8 && (((int64_t)units * split < sms && L.max_B / (2 * split) >= 64) ||
                       (L.max_B + split - 1) / split > kMaxChunk))
    split *= 2;
  c->split = split;
  c->stages = 0;
  c->prefill_path = 0;
  c->chunk_path = 0;
  c->decode_path = 0;
  {
    double sum = 0.0;
    for (int s2 = 0; s2 < cfg->batch; ++s2) sum += (double)cfg->heavy_budget[s2] + cfg->recent_window[s2];
    c->mean_budget = sum / cfg->batch;
  }
  c->chunk = (((L.max_B + split - 1) / split) + 3) & ~3;

  char* ws = static_cast<char*>(dev_workspace);
  h2o::CacheView& v = c->view;
  v.K = ws + L.K;
  v.V = ws + L.V;
  v.acc = reinterpret_cast<double*>(ws + L.acc);
  v.pos = reinterpret_cast<int32_t*>(ws + L.pos);
  v.count = reinterpret_cast<int32_t*>(ws + L.count);
  v.tpos = reinterpret_cast<int32_t*>(ws + L.tpos);
  v.status = reinterpret_cast<int32_t*>(ws + L.status);
  v.meta = reinterpret_cast<const h2o::UnitMeta*>(ws + L.meta);
  v.units = units;
  v.n_heads = cfg->n_heads;
  v.head_dim = cfg->head_dim;
  v.scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  {
    bool uniform = true;
    for (int s = 1; s < cfg->batch; ++s)
      uniform = uniform && c->heavy[s] == c->heavy[0] && c->recent[s] == c->recent[0];
    v.uni_pad = uniform ? ((c->heavy[0] + c->recent[0] + 3) & ~3) : -1;
    v.uni_k = c->heavy[0];
    v.uni_r = c->recent[0];
  }
  v.score_mode = 0;
  v.kv4 = cfg->dtype == H2O_BF16_KV4 ? 1 : 0;
  v.mask_kind = 0;
  v.mask_a = 1;
  v.mask_b = 0;
  v.topk = 0;
  v.seq_rwin = reinterpret_cast<const int32_t*>(ws + L.seq_rwin);
  v.total_slots = L.total_slots;
  v.group = group_of(cfg);
  c->seen.assign(cfg->batch, attach ? -1 : 0);

  bool ok = true;
  if (attach) {
    // the workspace already holds a cache: its unit table must be the one this configuration produces
    std::vector<h2o::UnitMeta> have(units);
    ok = cudaMemcpy(have.data(), ws + L.meta, units * sizeof(h2o::UnitMeta), cudaMemcpyDeviceToHost) == cudaSuccess;
    if (ok && std::memcmp(have.data(), meta.data(), units * sizeof(h2o::UnitMeta)) != 0) {
      delete c;
      return H2O_ERR_STATE;
    }
    c->phase = Phase::Decoding;  // whatever it holds, it is not to be prefilled again
  } else {
    ok = ok && cudaMemset(ws + L.acc, 0, L.meta - L.acc) == cudaSuccess;  // acc, pos, count, tpos, status
    ok = ok && cudaMemset(ws + L.pos, 0xff, (size_t)L.total_slots * sizeof(int32_t)) == cudaSuccess;  // pos = -1
    ok = ok && cudaMemcpy(ws + L.meta, meta.data(), units * sizeof(h2o::UnitMeta), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(ws + L.seq_rwin, c->recent.data(), (size_t)cfg->batch * sizeof(int32_t), cudaMemcpyHostToDevice) == cudaSuccess;
    // The memsets are asynchronous and a pageable copy returns once the data is staged, all on the legacy default
    // stream, which a non-blocking stream is not ordered behind: wait here, so that the tables are on the device
    // whatever stream the caller uses next.
    ok = ok && cudaStreamSynchronize(0) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    delete c;
    return H2O_ERR_CUDA;
  }
  *out = c;
  return H2O_OK;
}

int h2o_cache_create(h2o_cache_t** out, const h2o_config_t* cfg, void* dev_workspace, size_t workspace_bytes) {
  return create_impl(out, cfg, dev_workspace, workspace_bytes, false);
}

int h2o_cache_attach(h2o_cache_t** out, const h2o_config_t* cfg, void* dev_workspace, size_t workspace_bytes) {
  return create_impl(out, cfg, dev_workspace, workspace_bytes, true);
}

int h2o_prefill_select(h2o_cache_t* cache, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                       void* out, void* scratch, size_t scratch_bytes, void* stream) {
  if (!cache || !q || !k || !v || !cu_seqlens || !out || !scratch) return H2O_ERR_INVALID_ARG;
  if (cache->phase != Phase::Empty) return H2O_ERR_STATE;
  const h2o_config_t& cfg = cache->cfg;
  if (cu_seqlens[0] != 0) return H2O_ERR_INVALID_ARG;
  int max_seqlen = 0;
  for (int s = 0; s < cfg.batch; ++s) {
    const int64_t n = (int64_t)cu_seqlens[s + 1] - cu_seqlens[s];
    if (n < 1) return H2O_ERR_INVALID_ARG;
    max_seqlen = std::max<int64_t>(max_seqlen, n);
  }
  const int64_t total = cu_seqlens[cfg.batch];
  if (max_seqlen > kMaxPromptLen) return H2O_ERR_UNSUPPORTED;  // limit of the shared-memory score row
  const ScratchLayout S = make_scratch_layout(&cfg, total);
  if (scratch_bytes < S.total || (reinterpret_cast<uintptr_t>(scratch) % kAlign) != 0) return H2O_ERR_WORKSPACE;
  for (const void* p : {q, k, v, (const void*)out})
    if (reinterpret_cast<uintptr_t>(p) % 16 != 0) return H2O_ERR_INVALID_ARG;
  if (out == q || out == k || out == v) return H2O_ERR_INVALID_ARG;

  DeviceGuard guard(cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* sc = static_cast<char*>(scratch);
  h2o::PrefillScratch ps;
  ps.rowmax = reinterpret_cast<float*>(sc + S.rowstat);
  ps.rowsum = ps.rowmax + (size_t)total * cfg.n_heads * cache->view.group;
  ps.rowstat = reinterpret_cast<float2*>(sc + S.rowstat);
  ps.acc0 = reinterpret_cast<double*>(sc + S.acc0);
  ps.cu = reinterpret_cast<int32_t*>(sc + S.cu);
  ps.work = ps.cu + cfg.batch + 1;
  ps.total_tokens = total;
  cache->cu.assign(cu_seqlens, cu_seqlens + cfg.batch + 1);  // pageable source: staged before the call returns
  cache->cu.resize((size_t)cfg.batch + 3, 0);  // the work counters travel with it: zero at every launch
  ps.item_base = ps.cu + cfg.batch + 3;
  // (the forward kernels work on QUERY heads: with grouped-query attention a unit there is one query head)
  const int q_heads = cfg.n_heads * cache->view.group, q_units = cache->view.units * cache->view.group;
  ps.fs_grp = h2o::fwd_group_units(q_units, max_seqlen);
  ps.fs_groups = 0;
  ps.fs_items = 0;
  if (ps.fs_grp > 0) {  // item order of the persistent forward kernel: a group has as many levels as its longest
                        // sequence has query blocks of 128
    const int units = q_units, grp = ps.fs_grp;
    ps.fs_groups = (units + grp - 1) / grp;
    int64_t base = 0;
    cache->cu.push_back(0);
    for (int g = 0; g < ps.fs_groups; ++g) {
      const int u0 = g * grp, u1 = std::min(units, u0 + grp);
      int nbmax = 0;
      for (int sq = u0 / q_heads; sq <= (u1 - 1) / q_heads; ++sq)
        nbmax = std::max(nbmax, (int)(((int64_t)cu_seqlens[sq + 1] - cu_seqlens[sq] + 127) / 128));
      base += (int64_t)(u1 - u0) * nbmax;
      if (base > INT32_MAX) return H2O_ERR_UNSUPPORTED;
      cache->cu.push_back((int32_t)base);
    }
    ps.fs_items = (int32_t)base;
  }
  if (cudaMemcpyAsync(ps.cu, cache->cu.data(), cache->cu.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st) !=
      cudaSuccess) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  // bf16 / head_dim 128 runs on the tensor cores; every other combination on the fp32 FMA pipe
  const int in_dtype = input_dtype(cfg.dtype);
  // (a sparse pattern is applied by the fp32-FMA kernels only)
  const bool tc = cache->prefill_path != 1 && cache->view.mask_kind == 0 && h2o::prefill_tc_supported(in_dtype, cfg.head_dim);
  cudaError_t e = cudaSuccess;
  // optional phase events of this one call (diagnostic): before the forward kernel, after it, after the column
  // sums, after selection and gather
  cudaEvent_t pev[4];
  for (int i = 0; i < 4; ++i) {
    pev[i] = cache->prefill_events[i];
    cache->prefill_events[i] = nullptr;
  }
  auto stamp = [&](int i) {
    if (e == cudaSuccess && pev[i]) e = cudaEventRecord(pev[i], st);
  };
  stamp(0);
  if (tc) {
    if (e == cudaSuccess) e = h2o::launch_fwd_tc(cache->view, ps, max_seqlen, q, k, v, out, st);
    stamp(1);
    if (e == cudaSuccess) e = h2o::launch_colsum_tc(cache->view, ps, max_seqlen, q, k, st);
    stamp(2);
  } else {
    if (e == cudaSuccess) e = h2o::launch_prefill_naive(cache->view, ps, in_dtype, max_seqlen, q, k, v, out, true, false, st);
    stamp(1);
    if (e == cudaSuccess) e = h2o::launch_prefill_naive(cache->view, ps, in_dtype, max_seqlen, q, k, v, out, false, true, st);
    stamp(2);
  }
  if (e == cudaSuccess) e = h2o::launch_select_gather(cache->view, ps, in_dtype, std::min(cache->layout.max_B, max_seqlen), max_seqlen, k, v, st);
  if (e == cudaSuccess && cache->view.kv4) e = h2o::launch_gather_kv4(cache->view, ps, k, v, st);
  stamp(3);
  if (e != cudaSuccess) {
    // earlier kernels of this call may already be enqueued and have written part of the workspace
    cudaGetLastError();
    g_last_writer.note_and_check(st, cache->view.K);
    cache->phase = Phase::Failed;
    return H2O_ERR_CUDA;
  }
  g_last_writer.note_and_check(st, cache->view.K);  // select/gather wrote this cache
  for (int s = 0; s < cfg.batch; ++s) cache->seen[s] = (int64_t)cu_seqlens[s + 1] - cu_seqlens[s];
  cache->phase = Phase::Prefilled;
  return H2O_OK;
}

namespace {
// Which kernel serves a multi-head decode step.  The two-pass streaming kernel (K stream with the scores on
// mma.sync and the softmax statistics kept alongside, V stream; decode_two_pass.cu with one query head per unit) is
// the faster one for launches of more than two blocks per SM unless the units are small.  Per launch, online-softmax
// kernel against two-pass kernel: 4096 ragged units of 26..820 slots 148 / 140 us; 3584 units of 104 slots
// 44.4 / 42.2; 2048 units of 64 / 96 / 128 / 160 / 256 slots 18.3 / 19.6, 23.6 / 24.0, 28.0 / 27.4, 34.0 / 33.4,
// 54.5 / 47.1; 600 units of 128 / 300 slots 13.9 / 8.7, 23.6 / 17.2; 4096 units of 64 slots 34.0 / 38.8 us.  On
// 256 units of 410 slots both take 12.2 us, on 32 units of 2048 slots split over clusters of eight 11.3 - 12.0
// against 11.4: the online kernel stays there.
bool two_pass_supported(const h2o_cache* cache) {
  return cache->view.group == 1 && !cache->view.kv4 && (cache->view.topk == 0 || cache->split == 1) &&
         h2o::decode_two_pass_supported(cache->cfg.dtype, cache->cfg.head_dim, 1, cache->chunk);
}
bool two_pass_step(const h2o_cache* cache) {
  if (cache->decode_path == 1 || !two_pass_supported(cache)) return false;
  if (cache->decode_path == 2) return true;
  // "Top-K" attention: the selection's block barriers weigh differently on the two kernels: 256 units of 410 slots
  // 24.0 us on the online kernel's instance against 19.4 here, 4096 ragged units 170 against 180 us
  if (cache->view.topk > 0) return cache->view.units <= 2 * h2o::sm_count();
  return cache->split == 1 && cache->view.units > 2 * h2o::sm_count() && cache->mean_budget >= 100.0;
}
}  // namespace

int h2o_decode_step(h2o_cache_t* cache, const void* q, const void* k_new, const void* v_new, void* out,
                    int32_t* evicted_pos, void* stream) {
  if (!cache || !q || !k_new || !v_new || !out) return H2O_ERR_INVALID_ARG;
  if (cache->phase == Phase::Failed) return H2O_ERR_STATE;
  for (const void* p : {q, k_new, v_new, (const void*)out})
    if (reinterpret_cast<uintptr_t>(p) % 16 != 0) return H2O_ERR_INVALID_ARG;
  DeviceGuard guard(cache->cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  // the cache workspace is the identity: two handles on one workspace must count as the same cache
  const bool quiescent = g_last_writer.note_and_check(static_cast<cudaStream_t>(stream), cache->view.K) && g_early_prefetch;
  const bool ring1 = two_pass_step(cache);
  const cudaError_t e =
      ring1 ? h2o::launch_decode_two_pass(cache->view, cache->split, cache->chunk, quiescent, all_units_full(cache), q, k_new, v_new, out,
                                          evicted_pos, static_cast<cudaStream_t>(stream))
      : cache->view.group > 1
          ? h2o::launch_decode_gqa(cache->view, cache->cfg.dtype, cache->layout.max_B, quiescent, all_units_full(cache), q, k_new,
                                   v_new, out, evicted_pos, static_cast<cudaStream_t>(stream))
      : cache->view.kv4 ? h2o::launch_decode_kv4(cache->view, cache->split, cache->chunk, quiescent, all_units_full(cache), q, k_new,
                                               v_new, out, evicted_pos, static_cast<cudaStream_t>(stream))
                      : h2o::launch_decode(cache->view, cache->cfg.dtype, cache->split, cache->chunk, cache->stages, quiescent,
                                           all_units_full(cache), q, k_new, v_new, out, evicted_pos,
                                           static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  advance_seen(cache, 1);
  cache->phase = Phase::Decoding;
  return H2O_OK;
}

int h2o_decode_chunk(h2o_cache_t* cache, const void* q, const void* k, const void* v, int32_t n_tokens, void* out,
                     int32_t* evicted_pos, void* stream) {
  if (!cache || !q || !k || !v || !out || n_tokens < 1) return H2O_ERR_INVALID_ARG;
  if (cache->phase == Phase::Failed) return H2O_ERR_STATE;
  for (const void* p : {q, k, v, (const void*)out})
    if (reinterpret_cast<uintptr_t>(p) % 16 != 0) return H2O_ERR_INVALID_ARG;
  DeviceGuard guard(cache->cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  g_last_writer.note_and_check(st, cache->view.K);
  cudaError_t e = cudaSuccess;
  // (the chunk kernel ranks by the accumulated score only)
  if (cache->chunk_path == 0 && cache->view.score_mode == 0 && cache->view.mask_kind == 0 && cache->view.topk == 0 &&
      cache->view.group == 1 && !cache->view.kv4 && h2o::decode_chunk_supported(cache->cfg.dtype, cache->cfg.head_dim, cache->layout.max_B,
                                                          cache->layout.total_slots)) {
    e = h2o::launch_decode_chunk(cache->view, cache->layout.total_slots, cache->meta.data(), q, k, v, n_tokens, out,
                                 evicted_pos, st);
    if (e == cudaSuccess) advance_seen(cache, n_tokens);
  } else {
    const size_t step = (size_t)cache->view.units * cache->cfg.head_dim * elem_size(cache->cfg.dtype);
    const size_t qstep = step * cache->view.group;  // q and out carry the group's query heads
    for (int32_t i = 0; i < n_tokens && e == cudaSuccess; ++i) {
      const size_t off = (size_t)i * step;
      int32_t* ev_i = evicted_pos ? evicted_pos + (size_t)i * cache->view.units : nullptr;
      e = cache->view.group > 1
              ? h2o::launch_decode_gqa(cache->view, cache->cfg.dtype, cache->layout.max_B, false, all_units_full(cache),
                                       static_cast<const char*>(q) + i * qstep,
                                       static_cast<const char*>(k) + off, static_cast<const char*>(v) + off,
                                       static_cast<char*>(out) + i * qstep, ev_i, st)
          : two_pass_step(cache)
              ? h2o::launch_decode_two_pass(cache->view, cache->split, cache->chunk, false, all_units_full(cache),
                                            static_cast<const char*>(q) + off, static_cast<const char*>(k) + off,
                                            static_cast<const char*>(v) + off, static_cast<char*>(out) + off, ev_i, st)
          : cache->view.kv4
              ? h2o::launch_decode_kv4(cache->view, cache->split, cache->chunk, false, all_units_full(cache), static_cast<const char*>(q) + off,
                                       static_cast<const char*>(k) + off, static_cast<const char*>(v) + off,
                                       static_cast<char*>(out) + off, ev_i, st)
              : h2o::launch_decode(cache->view, cache->cfg.dtype, cache->split, cache->chunk, cache->stages, false,
                                   all_units_full(cache), static_cast<const char*>(q) + off, static_cast<const char*>(k) + off,
                                   static_cast<const char*>(v) + off, static_cast<char*>(out) + off, ev_i, st);
      if (e == cudaSuccess) advance_seen(cache, 1);
    }
  }
  if (e != cudaSuccess) {
    // some of the tokens may already have been enqueued: the cache no longer matches what the caller knows
    cudaGetLastError();
    cache->phase = Phase::Failed;
    return H2O_ERR_CUDA;
  }
  cache->phase = Phase::Decoding;
  return H2O_OK;
}

int h2o_cache_set_score_mode(h2o_cache_t* cache, int32_t mode) {
  if (!cache || (mode != 0 && mode != 1)) return H2O_ERR_INVALID_ARG;
  if (cache->phase != Phase::Empty) return H2O_ERR_STATE;  // one ranking rule per generation
  cache->view.score_mode = mode;
  return H2O_OK;
}

int h2o_cache_set_mask(h2o_cache_t* cache, int32_t kind, int32_t a, int32_t b) {
  if (!cache || kind < 0 || kind > 2) return H2O_ERR_INVALID_ARG;
  if (kind != 0 && (a < 1 || b < 0 || (kind == 2 && b > a))) return H2O_ERR_INVALID_ARG;
  if (cache->phase != Phase::Empty) return H2O_ERR_STATE;  // one attention rule per generation
  // (4-bit slots have no pattern form; of the grouped step kernels the streaming one applies patterns)
  if (kind != 0 && (cache->view.kv4 || (cache->view.group > 1 &&
                                        !h2o::decode_two_pass_supported(cache->cfg.dtype, cache->cfg.head_dim, cache->view.group,
                                                                        cache->layout.max_B))))
    return H2O_ERR_UNSUPPORTED;
  cache->view.mask_kind = kind;
  cache->view.mask_a = kind ? a : 1;
  cache->view.mask_b = kind ? b : 0;
  return H2O_OK;
}

int h2o_cache_set_topk(h2o_cache_t* cache, int32_t m) {
  if (!cache || m < 0) return H2O_ERR_INVALID_ARG;
  if (cache->phase != Phase::Empty) return H2O_ERR_STATE;  // one attention rule per generation
  if (m > 0) {
    if (cache->view.kv4 || cache->view.group > 1) return H2O_ERR_UNSUPPORTED;
    const int chunk = (cache->layout.max_B + 3) & ~3;  // one thread block per unit: the selection runs over its scores
    if (chunk > kMaxChunk) return H2O_ERR_UNSUPPORTED;
    cache->split = 1;
    cache->chunk = chunk;
  }
  cache->view.topk = m;
  return H2O_OK;
}

int h2o_cache_fscore(h2o_cache_t* cache, int32_t hkind, double* out_dev, void* stream) {
  if (!cache || !out_dev || hkind < 0 || hkind > 2) return H2O_ERR_INVALID_ARG;
  DeviceGuard guard(cache->cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  if (h2o::launch_fscore(cache->view, hkind, out_dev, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  return H2O_OK;
}

int h2o_cache_set_decode_path(h2o_cache_t* cache, int32_t path) {
  if (!cache || path < 0 || path > 2) return H2O_ERR_INVALID_ARG;
  if (path == 2 && !two_pass_supported(cache)) return H2O_ERR_UNSUPPORTED;
  cache->decode_path = path;
  return H2O_OK;
}

int h2o_cache_get_decode_path(h2o_cache_t* cache) {
  if (!cache) return H2O_ERR_INVALID_ARG;
  if (cache->view.group > 1)
    return h2o::decode_two_pass_supported(cache->cfg.dtype, cache->cfg.head_dim, cache->view.group, cache->layout.max_B) ? 2 : 1;
  return two_pass_step(cache) ? 2 : 1;
}

int h2o_cache_set_chunk_path(h2o_cache_t* cache, int32_t path) {
  if (!cache || (path != 0 && path != 1)) return H2O_ERR_INVALID_ARG;
  cache->chunk_path = path;
  return H2O_OK;
}

size_t h2o_host_staging_bytes(const h2o_config_t* cfg, int64_t tokens) {
  if (check_config(cfg) != H2O_OK || tokens < 1 || tokens > INT32_MAX) return 0;
  const size_t kv = align_up((size_t)tokens * cfg->n_heads * cfg->head_dim * elem_size(cfg->dtype));
  const size_t qo = align_up((size_t)tokens * cfg->n_heads * group_of(cfg) * cfg->head_dim * elem_size(cfg->dtype));
  return 2 * qo + 2 * kv + align_up((size_t)tokens * cfg->n_heads * sizeof(int32_t));  // q, k, v, out, evicted
}

int h2o_prefill_select_host(h2o_cache_t* cache, const void* q_host, const void* k_host, const void* v_host,
                            const int32_t* cu_seqlens, void* out_host, void* staging, size_t staging_bytes,
                            void* scratch, size_t scratch_bytes, void* stream) {
  if (!cache || !q_host || !k_host || !v_host || !cu_seqlens || !out_host || !staging) return H2O_ERR_INVALID_ARG;
  if (cache->phase != Phase::Empty) return H2O_ERR_STATE;
  const h2o_config_t& cfg = cache->cfg;
  const int64_t total = cu_seqlens[cfg.batch];
  if (total < 1) return H2O_ERR_INVALID_ARG;
  if (staging_bytes < h2o_host_staging_bytes(&cfg, total) || (reinterpret_cast<uintptr_t>(staging) % kAlign) != 0)
    return H2O_ERR_WORKSPACE;
  DeviceGuard guard(cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // staging: q | k | v | out; with grouped-query attention q and out carry n_heads * group heads
  const size_t bytes = (size_t)total * cfg.n_heads * cfg.head_dim * elem_size(cfg.dtype);
  const size_t qbytes = bytes * cache->view.group;
  const size_t pitch = align_up(bytes), qpitch = align_up(qbytes);
  char* sg = static_cast<char*>(staging);
  char *sq = sg, *sk = sg + qpitch, *sv = sk + pitch, *so = sv + pitch;
  bool ok = cudaMemcpyAsync(sq, q_host, qbytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(sk, k_host, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(sv, v_host, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  const int rc = h2o_prefill_select(cache, sq, sk, sv, cu_seqlens, so, scratch, scratch_bytes, stream);
  if (rc != H2O_OK) return rc;
  if (cudaMemcpyAsync(out_host, so, qbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  return H2O_OK;
}

int h2o_decode_step_host(h2o_cache_t* cache, const void* q_host, const void* k_new_host, const void* v_new_host,
                         void* out_host, int32_t* evicted_pos_host, void* staging, size_t staging_bytes, void* stream) {
  if (!cache || !q_host || !k_new_host || !v_new_host || !out_host || !staging) return H2O_ERR_INVALID_ARG;
  const h2o_config_t& cfg = cache->cfg;
  if (staging_bytes < h2o_host_staging_bytes(&cfg, cfg.batch) || (reinterpret_cast<uintptr_t>(staging) % kAlign) != 0)
    return H2O_ERR_WORKSPACE;
  DeviceGuard guard(cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)cfg.batch * cfg.n_heads * cfg.head_dim * elem_size(cfg.dtype);
  const size_t qbytes = bytes * cache->view.group;  // q and out carry n_heads * group heads
  const size_t pitch = align_up(bytes), qpitch = align_up(qbytes);
  char* sg = static_cast<char*>(staging);
  char *sq = sg, *sk = sg + qpitch, *sv = sk + pitch, *so = sv + pitch;
  int32_t* ev_dev = reinterpret_cast<int32_t*>(so + qpitch);
  // Pinned (or registered) host memory is addressable by the device: a decode step moves only a few
  // hundred bytes per unit, so the kernel reads its inputs and writes its results straight over the
  // bus instead of paying five small copies around every launch.  Pageable buffers take the copies.
  {
    void* dq = device_alias(q_host);
    void* dk = device_alias(k_new_host);
    void* dv = device_alias(v_new_host);
    void* dout = device_alias(out_host);
    void* dev_ev = evicted_pos_host ? device_alias(evicted_pos_host) : nullptr;
    if (dq && dk && dv && dout && (!evicted_pos_host || dev_ev))
      return h2o_decode_step(cache, dq, dk, dv, dout, static_cast<int32_t*>(dev_ev), stream);
  }
  bool ok = cudaMemcpyAsync(sq, q_host, qbytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(sk, k_new_host, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(sv, v_new_host, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  const int rc = h2o_decode_step(cache, sq, sk, sv, so, evicted_pos_host ? ev_dev : nullptr, stream);
  if (rc != H2O_OK) return rc;
  ok = cudaMemcpyAsync(out_host, so, qbytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (evicted_pos_host)
    ok = ok && cudaMemcpyAsync(evicted_pos_host, ev_dev, (size_t)cfg.batch * cfg.n_heads * sizeof(int32_t),
                               cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  return H2O_OK;
}

int h2o_cache_reset(h2o_cache_t* cache, void* stream) {
  if (!cache) return H2O_ERR_INVALID_ARG;
  DeviceGuard guard(cache->cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Layout& L = cache->layout;
  char* ws = static_cast<char*>(cache->view.K) - L.K;
  bool ok = cudaMemsetAsync(ws + L.acc, 0, L.meta - L.acc, st) == cudaSuccess;
  ok = ok && cudaMemsetAsync(ws + L.pos, 0xff, (size_t)L.total_slots * sizeof(int32_t), st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  g_last_writer.note_and_check(st, cache->view.K);  // the memsets wrote this cache
  cache->seen.assign(cache->cfg.batch, 0);
  cache->phase = Phase::Empty;
  return H2O_OK;
}

int h2o_cache_set_decode_shape(h2o_cache_t* cache, int32_t split, int32_t stages) {
  if (!cache || stages < 0 || stages > 8) return H2O_ERR_INVALID_ARG;
  if (split != 0 && split != 1 && split != 2 && split != 4 && split != 8) return H2O_ERR_INVALID_ARG;
  if (split > 1 && cache->view.topk > 0) return H2O_ERR_UNSUPPORTED;  // "Top-K" attention keeps a unit in one block
  if (split != 0) {
    const int chunk = (((cache->layout.max_B + split - 1) / split) + 3) & ~3;
    if (chunk > kMaxChunk) return H2O_ERR_UNSUPPORTED;
    cache->split = split;
    cache->chunk = chunk;
  }
  cache->stages = stages;
  return H2O_OK;
}

int h2o_cache_set_prefill_path(h2o_cache_t* cache, int32_t path) {
  if (!cache || (path != 0 && path != 1)) return H2O_ERR_INVALID_ARG;
  cache->prefill_path = path;
  return H2O_OK;
}

int h2o_prefill_scratch_layout(const h2o_config_t* cfg, int64_t total_tokens, size_t* acc0_offset) {
  if (check_config(cfg) != H2O_OK || total_tokens < 1 || total_tokens > INT32_MAX) return H2O_ERR_INVALID_ARG;
  const ScratchLayout S = make_scratch_layout(cfg, total_tokens);
  if (acc0_offset) *acc0_offset = S.acc0;
  return H2O_OK;
}

int h2o_debug_set_prefill_events(h2o_cache_t* cache, void* const* events) {
  if (!cache) return H2O_ERR_INVALID_ARG;
  for (int i = 0; i < 4; ++i) cache->prefill_events[i] = events ? static_cast<cudaEvent_t>(events[i]) : nullptr;
  return H2O_OK;
}

int h2o_debug_set_early_prefetch(int32_t enabled) {
  const int prev = g_early_prefetch ? 1 : 0;
  g_early_prefetch = enabled != 0;
  return prev;
}

int h2o_cache_destroy(h2o_cache_t* cache) {
  if (cache) g_last_writer.forget(cache->view.K);
  delete cache;
  return H2O_OK;
}

int h2o_cache_export(h2o_cache_t* cache, int32_t* pos, double* acc, int32_t* count, int32_t* t, int32_t pitch,
                     void* stream) {
  if (!cache) return H2O_ERR_INVALID_ARG;
  if ((pos || acc) && pitch < cache->layout.max_B) return H2O_ERR_INVALID_ARG;
  DeviceGuard guard(cache->cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const h2o::CacheView& v = cache->view;
  const size_t slots = (size_t)cache->layout.total_slots;
  std::vector<int32_t> hpos(pos ? slots : 0);
  std::vector<double> hacc(acc ? slots : 0);
  bool ok = cudaStreamSynchronize(st) == cudaSuccess;
  if (pos) ok = ok && cudaMemcpy(hpos.data(), v.pos, slots * sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess;
  if (acc) ok = ok && cudaMemcpy(hacc.data(), v.acc, slots * sizeof(double), cudaMemcpyDeviceToHost) == cudaSuccess;
  std::vector<int32_t> hcount(count ? v.units : 0), ht(t ? v.units : 0);
  if (count) ok = ok && cudaMemcpy(hcount.data(), v.count, v.units * sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess;
  if (t) ok = ok && cudaMemcpy(ht.data(), v.tpos, v.units * sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  for (int su = 0; su < v.units; ++su) {  // device tables are in launch order
    const h2o::UnitMeta& mt = cache->meta[su];
    const int u = mt.unit, B = mt.kbud + mt.rwin;
    for (int x = 0; x < pitch; ++x) {
      if (pos) pos[(size_t)u * pitch + x] = x < B ? hpos[mt.slot_off + x] : -1;
      if (acc) acc[(size_t)u * pitch + x] = x < B ? hacc[mt.slot_off + x] : 0.0;
    }
    if (count) count[u] = hcount[su];
    if (t) t[u] = ht[su];
  }
  return H2O_OK;
}

int h2o_cache_status(h2o_cache_t* cache, void* stream) {
  if (!cache) return H2O_ERR_INVALID_ARG;
  DeviceGuard guard(cache->cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  int32_t word = 0;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess ||
      cudaMemcpy(&word, cache->view.status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  return word;
}

int h2o_debug_wait_probe(h2o_cache_t* cache, int32_t polls, void* stream) {
  if (!cache || polls < 1 || polls > (1 << 20)) return H2O_ERR_INVALID_ARG;
  DeviceGuard guard(cache->cfg.device);
  if (!guard.ok) return H2O_ERR_CUDA;
  if (h2o::launch_wait_probe(cache->view, (uint32_t)polls, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return H2O_ERR_CUDA;
  }
  return H2O_OK;
}

int h2o_debug_bounds_checked(void) {
#ifdef H2O_BOUNDS
  return 1;
#else
  return 0;
#endif
}

const char* h2o_strerror(int code) {
  switch (code) {
    case H2O_OK: return "ok";
    case H2O_ERR_INVALID_ARG: return "invalid argument";
    case H2O_ERR_UNSUPPORTED: return "unsupported dtype, head_dim, size or device";
    case H2O_ERR_WORKSPACE: return "workspace or scratch too small or misaligned";
    case H2O_ERR_STATE: return "call order violated or inconsistent cache state";
    case H2O_ERR_CUDA: return "CUDA runtime error";
    case H2O_ERR_TIMEOUT: return "bounded device-side wait timed out";
    default: return "unknown error";
  }
}

}  // extern "C"
