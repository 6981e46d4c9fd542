// C ABI of the spectral projection (Eq. 1): projector lifetime, argument checks, tensor maps, launch.
#include <new>

#include "twkv_dev.h"
#include "tc_util.cuh"

struct twkv_projector {
  int device = 0, sm_count = 0, d = 0, bf16 = 0;
  unsigned char* ws = nullptr;                 // [status, 256 B][U_k^T][U_v^T]
  bool has[2] = {false, false};
  CUtensorMap map_uT[2];                       // box = one slab of U^T rows (single-CTA kernel)
  CUtensorMap map_uT_half[2];                  // box = 128 rows (CTA-pair kernel: each CTA loads half a slab)
};

namespace twkv {
constexpr size_t PJ_STATUS_BYTES = 256;
constexpr int PJ_PAIR_MIN_TOKENS = 1024;      // from here on the CTA-pair kernel is used (d a multiple of 256)
static bool dim_ok(int d) { return d >= 128 && d <= 8192 && d % 128 == 0; }
}  // namespace twkv

using namespace twkv;

extern "C" {

size_t twkv_projector_required_bytes(int d_kv) {
  if (!dim_ok(d_kv)) return 0;
  return PJ_STATUS_BYTES + 2 * (size_t)d_kv * d_kv * 2;
}

twkv_status twkv_projector_create(int d_kv, twkv_dtype dtype, const void* U_k, const void* U_v, void* workspace,
                                  size_t workspace_bytes, void* stream, twkv_projector** out) {
  if (!out) return TWKV_ERR_INVALID_ARG;
  *out = nullptr;
  if (!dim_ok(d_kv) || (dtype != TWKV_F16 && dtype != TWKV_BF16)) return TWKV_ERR_UNSUPPORTED;
  if (!workspace || (!U_k && !U_v)) return TWKV_ERR_INVALID_ARG;
  if ((uintptr_t)workspace % 256 || ((uintptr_t)U_k | (uintptr_t)U_v) % 16) return TWKV_ERR_INVALID_ARG;
  if (workspace_bytes < twkv_projector_required_bytes(d_kv)) return TWKV_ERR_CAPACITY;
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, workspace) != cudaSuccess) { cudaGetLastError(); return TWKV_ERR_CUDA; }
  if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) return TWKV_ERR_INVALID_ARG;
  twkv_projector* p = new (std::nothrow) twkv_projector();
  if (!p) return TWKV_ERR_INVALID_ARG;
  p->device = attr.device; p->d = d_kv; p->bf16 = dtype == TWKV_BF16 ? 1 : 0; p->ws = (unsigned char*)workspace;
  DeviceGuard g(p->device);
  cudaStream_t st = (cudaStream_t)stream;
  bool ok = g.ok && cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device) == cudaSuccess &&
            cudaMemsetAsync(p->ws, 0, PJ_STATUS_BYTES, st) == cudaSuccess;
  const int NS = (d_kv % 256 == 0) ? 256 : 128;
  const void* U[2] = {U_k, U_v};
  for (int side = 0; side < 2 && ok; ++side) {
    if (!U[side]) continue;
    // K-major copy of U for the tensor cores: row n of the copy = column n of U
    unsigned char* dst = p->ws + PJ_STATUS_BYTES + (size_t)side * d_kv * d_kv * 2;
    ok = launch_transpose16(U[side], dst, d_kv, st) == cudaSuccess &&
         make_tmap_2d(&p->map_uT[side], dst, d_kv, d_kv, (uint64_t)d_kv * 2, NS) &&
         make_tmap_2d(&p->map_uT_half[side], dst, d_kv, d_kv, (uint64_t)d_kv * 2, TILE);
    p->has[side] = true;
  }
  if (!ok) { delete p; return TWKV_ERR_CUDA; }
  *out = p;
  return TWKV_OK;
}

void twkv_projector_destroy(twkv_projector* p) { delete p; }

twkv_status twkv_project(twkv_projector* p, const void* x_k, const void* x_v, void* xt_k, void* xt_v, int n_tok, void* stream) {
  if (!p || n_tok < 0) return TWKV_ERR_INVALID_ARG;
  if ((x_k == nullptr) != (xt_k == nullptr) || (x_v == nullptr) != (xt_v == nullptr)) return TWKV_ERR_INVALID_ARG;
  if ((x_k && !p->has[0]) || (x_v && !p->has[1])) return TWKV_ERR_INVALID_ARG;
  if (((uintptr_t)x_k | (uintptr_t)x_v | (uintptr_t)xt_k | (uintptr_t)xt_v) % 16) return TWKV_ERR_INVALID_ARG;
  if (n_tok == 0 || (!x_k && !x_v)) return TWKV_OK;
  const size_t bytes = (size_t)n_tok * p->d * 2;
  const void* in[2] = {x_k, x_v};
  void* outp[2] = {xt_k, xt_v};
  for (int i = 0; i < 2; ++i)
    for (int o = 0; o < 2; ++o)
      if (in[i] && outp[o] && (const unsigned char*)in[i] < (unsigned char*)outp[o] + bytes &&
          (unsigned char*)outp[o] < (const unsigned char*)in[i] + bytes) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(p->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  const int side0 = x_k ? 0 : 1, n_sides = (x_k ? 1 : 0) + (x_v ? 1 : 0);
  const bool pairs = p->d % 256 == 0 && n_tok >= PJ_PAIR_MIN_TOKENS && project_tc_max_pairs(p->sm_count) > 0;
  ProjectMaps maps;
  for (int side = 0; side < 2; ++side) {
    const int src = in[side] ? side : side0;              // an unused side's maps alias the used one (never dereferenced)
    CUtensorMap* mx = side ? &maps.xv : &maps.xk;
    CUtensorMap* mo = side ? &maps.ov : &maps.ok;
    if (!make_tmap_2d(mx, in[src], (uint64_t)n_tok, p->d, (uint64_t)p->d * 2, TILE) ||
        !make_tmap_2d(mo, outp[src], (uint64_t)n_tok, p->d, (uint64_t)p->d * 2, TILE)) return TWKV_ERR_CUDA;
    (side ? maps.uv : maps.uk) = pairs ? p->map_uT_half[src] : p->map_uT[src];
  }
  if (launch_project_tc(maps, n_tok, p->d, p->bf16, side0, n_sides, (int*)p->ws, p->sm_count, pairs, (cudaStream_t)stream) != cudaSuccess)
    return TWKV_ERR_CUDA;
  return TWKV_OK;
}

twkv_status twkv_projector_status(twkv_projector* p, void* stream) {
  if (!p) return TWKV_ERR_INVALID_ARG;
  DeviceGuard g(p->device);
  if (!g.ok) return TWKV_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  int code = 0;
  if (cudaMemcpyAsync(&code, p->ws, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TWKV_ERR_CUDA;
  if (code != 0) {
    if (cudaMemsetAsync(p->ws, 0, sizeof(int), st) != cudaSuccess) return TWKV_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TWKV_ERR_CUDA;
  }
  return (twkv_status)code;
}

}  // extern "C"
