// h2o_prefill_select_static: prefill-select for callers that must not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits — a plugin called from inside
// somebody else's serving loop that owns the whole memory pool, a latency-critical path that
// may not take the allocator's lock or its implicit synchronisation, an embedding in a runtime
// that hands out device memory only at start-up.  Such a caller can pass inputs and outputs it
// already owns, but has nowhere to get the scratch buffer h2o_prefill_select asks for.
//
// Here the scratch lives in a fixed array inside the library image.  Every GPU that loads the
// library carries the array (kStaticScratchBytes) until the process exits, whether or not this
// entry point is ever called, so the size is kept modest and prompts that need more are refused.
#include <mutex>

#include "h2o_internal.cuh"

namespace {

constexpr size_t kStaticScratchBytes = (size_t)16 << 20;  // 16 MiB: about one million (token, head) cells
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a stand-in for the symbol, NOT a device
// address: handing it to a kernel would fault (or, where the GPU can reach host memory, quietly
// use the wrong bytes).  Host code must ask the runtime for the address — see scratch_address().
static __device__ __align__(256) unsigned char g_prefill_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void* g_scratch_address[kMaxDevices] = {};  // per device: where the array lives there (nullptr = not asked yet)

// Device address of the array on `device`; looked up once per device with that device current.
int scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return H2O_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_address[device]) {
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) {
      cudaGetLastError();
      return H2O_ERR_CUDA;
    }
    if (prev != device && cudaSetDevice(device) != cudaSuccess) {
      cudaGetLastError();
      return H2O_ERR_CUDA;
    }
    void* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&ptr, g_prefill_scratch);
    if (prev != device) cudaSetDevice(prev);
    if (e != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return H2O_ERR_CUDA;
    }
    g_scratch_address[device] = ptr;
  }
  *out = g_scratch_address[device];
  return H2O_OK;
}

}  // namespace

extern "C" {

size_t h2o_prefill_static_scratch_bytes(void) { return kStaticScratchBytes; }

int h2o_prefill_select_static(h2o_cache_t* cache, const void* q, const void* k, const void* v,
                              const int32_t* cu_seqlens, void* out, void* stream) {
  if (!cache || !cu_seqlens) return H2O_ERR_INVALID_ARG;
  const h2o_config_t* cfg = h2o::cache_config(cache);
  const int64_t total = cu_seqlens[cfg->batch];
  const size_t need = h2o_prefill_scratch_bytes(cfg, total);
  if (need == 0) return H2O_ERR_INVALID_ARG;
  if (need > kStaticScratchBytes) return H2O_ERR_WORKSPACE;  // prompt too large for the built-in scratch
  void* scratch = nullptr;
  const int rc = scratch_address(cfg->device, &scratch);
  if (rc != H2O_OK) return rc;
  // Same kernels, same order, same stream semantics as the caller-scratch entry point.  Nothing in
  // the scratch has to start at zero: every cell that is read was written earlier in the same call.
  return h2o_prefill_select(cache, q, k, v, cu_seqlens, out, scratch, kStaticScratchBytes, stream);
}

}  // extern "C"
