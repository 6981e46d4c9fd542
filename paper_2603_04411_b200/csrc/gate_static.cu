// twkv_gate_ranks_static: the gate (logits GEMM -> softmax -> cumsum -> threshold) for a small
// batch of tokens, with its logits scratch in a fixed device array instead of caller memory.
//
// Why it exists.  Every other entry point of this library keeps its scratch inside the pool the
// caller handed to twkv_cache_create.  Some callers want the ranks of a handful of new tokens
// before they own such a pool, and cannot obtain device memory themselves: a request scheduler
// that budgets cache blocks from the predicted ranks, code running inside a serving loop whose
// framework has reserved the whole device and forbids raw allocations, or a latency-critical
// path that must not take the device-wide synchronisation an allocation can imply.  For them
// the scratch lives in the library image.
//
// Cost and limits.  The array below is 4 MiB and is resident on every GPU that loads the
// library, until the process exits.  It holds the fp32 logits of at most
// TWKV_STATIC_GATE_MAX_ROWS = 1024 (token, side) rows of width d_kv <= 1024, i.e. 512 tokens at
// d_kv = 1024.  All calls on a device share it and it keeps the previous call's logits: the
// GEMM overwrites every row it will read, so nothing has to be cleared, but two calls that
// overlap on the GPU (different streams, or different host threads) race on it.
#include <mutex>

#include "twkv_dev.h"

namespace twkv {

constexpr int STATIC_GATE_MAX_ELEMS = 1024 * 1024;          // 1024 rows x 1024 logits, fp32 = 4 MiB
static __device__ __align__(256) float g_static_gate_logits[STATIC_GATE_MAX_ELEMS];

// In host code the array's name is only a handle of the symbol, not a device address; the address
// has to be asked for once per device, with that device current.
constexpr int MAX_DEVICES = 64;
static std::mutex g_static_mu;
static float* g_static_ptr[MAX_DEVICES] = {nullptr};

static cudaError_t static_scratch(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_gate_logits);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_static_ptr[dev];
  return cudaSuccess;
}

}  // namespace twkv

using namespace twkv;

extern "C" twkv_status twkv_gate_ranks_static(const void* K, const void* V, const void* W_k, const void* W_v,
                                              const float* b_k, const float* b_v, int n_tok, int d_kv, int dtype,
                                              float tau, uint16_t* levels, void* stream) {
  if (n_tok < 0) return TWKV_ERR_INVALID_ARG;
  if (n_tok == 0) return TWKV_OK;
  if (!K || !V || !W_k || !W_v || !levels) return TWKV_ERR_INVALID_ARG;
  if (d_kv < 128 || d_kv > 1024 || d_kv % 128) return TWKV_ERR_UNSUPPORTED;
  if (dtype != TWKV_F16 && dtype != TWKV_BF16) return TWKV_ERR_UNSUPPORTED;
  if (!(tau > 0.f && tau < 1.f)) return TWKV_ERR_INVALID_ARG;
  if (((uintptr_t)K | (uintptr_t)V | (uintptr_t)W_k | (uintptr_t)W_v) % 16 || (uintptr_t)levels % 4) return TWKV_ERR_INVALID_ARG;
  if ((long long)n_tok * 2 * d_kv > (long long)STATIC_GATE_MAX_ELEMS) return TWKV_ERR_CAPACITY;   // beyond the fixed scratch
  float* scratch = nullptr;
  if (static_scratch(&scratch) != cudaSuccess) { cudaGetLastError(); return TWKV_ERR_CUDA; }
  DevView v{};                    // only the shape fields the two launchers read (no status word: v.status stays null)
  v.d_kv = d_kv; v.dtype = dtype; v.tau = tau;
  LayerParams lp{nullptr, nullptr, W_k, W_v, b_k, b_v};
  cudaStream_t st = (cudaStream_t)stream;
  if (launch_gate_logits(v, lp, K, V, n_tok, scratch, st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (launch_gate_rank(v, scratch, levels, n_tok, st) != cudaSuccess) return TWKV_ERR_CUDA;
  return TWKV_OK;
}
