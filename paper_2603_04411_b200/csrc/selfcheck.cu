// Diagnostics that are not part of the method: a consistency check of a cache's tables and guard words, and a
// self-test of the bounded device-side wait every tensor-core kernel of the library relies on.
#include "twkv_dev.h"
#include "tc_util.cuh"

namespace twkv {

// ------------------------------------------------------------------------------------------
// A wait nobody will end: the same mbar_wait the production kernels use, with its attempt limit given by the caller.
// The barrier is initialised for one arrival that never comes.  The kernel must give up, raise the CTA's abort flag
// like a production role does, and report TWKV_ERR_TIMEOUT through the status word; out[0..1] = elapsed nanoseconds
// (global timer), out[2] = 1 if the wait reported failure.
__global__ void __launch_bounds__(64) wait_timeout_kernel(DevView v, unsigned attempts, unsigned long long* out) {
  __shared__ __align__(8) unsigned long long bar_mem;
  __shared__ int abort_flag;
  const uint32_t bar = tc::smem_addr(&bar_mem);
  if (threadIdx.x == 0) {
    tc::mbar_init(bar, 1);
    abort_flag = 0;
    tc::mbar_init_fence();
  }
  __syncthreads();
  unsigned long long t0 = 0, t1 = 0;
  bool ok = true;
  if (threadIdx.x < 32) {
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    ok = tc::mbar_wait_limited(bar, 0u, &abort_flag, attempts);        // phase 0 never completes
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
  }
  __syncthreads();
  // the second warp polls the flag the way the other roles of a production kernel do
  if (threadIdx.x == 32) out[2] = (unsigned long long)(*(volatile int*)&abort_flag);
  if (threadIdx.x == 0) {
    out[0] = t1 - t0;
    out[1] = ok ? 0ull : 1ull;
    if (abort_flag) set_status(v, TWKV_ERR_TIMEOUT);
  }
}

cudaError_t launch_wait_timeout(const DevView& v, unsigned attempts, unsigned long long* out_dev, cudaStream_t st) {
  wait_timeout_kernel<<<1, 64, 0, st>>>(v, attempts, out_dev);
  count_launch();
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Table and guard check.  One CTA; every violation sets TWKV_ERR_DEVICE_CHECK (sticky) and counts in out[0].
//   - the guard words written behind every region of the pool at creation are intact
//   - per tile: sequence < S, 1 <= class <= NC, 0 <= n_valid <= 128, its blocks lie below the bump pointer
//   - per valid slot: 64 (class - 1) < rank <= 64 class; a V slot links to a valid slot of a K tile of the same sequence
//   - tile lists name tiles that exist, of the right class / sequence
__global__ void __launch_bounds__(1024) cache_check_kernel(DevView v, int l0, int l1, const unsigned long long* guards, int n_guards,
                                                          unsigned long long* out) {
  __shared__ unsigned s_bad;
  if (threadIdx.x == 0) s_bad = 0u;
  __syncthreads();
  unsigned bad = 0u;
  for (int i = threadIdx.x; i < n_guards; i += blockDim.x)
    if (*reinterpret_cast<const unsigned long long*>(reinterpret_cast<const unsigned char*>(v.status) + guards[i]) != TWKV_GUARD_WORD) ++bad;
  const int next_block = v.status[1];
  if (threadIdx.x == 0 && (next_block < 0 || next_block > v.n_blocks)) ++bad;
  for (int l = l0; l < l1; ++l) {
    for (int side = 0; side < 2; ++side) {
      const int nt = v.ntiles(l)[side];
      if (nt < 0 || nt > v.NT) { if (threadIdx.x == 0) ++bad; continue; }
      const int4* desc = v.desc(l, side);
      const int* aux = v.aux(l, side);
      const unsigned short* rank = v.rank(l, side);
      const int4* kdesc = v.desc(l, 0);
      const int ntk = v.ntiles(l)[0];
      for (long long i = threadIdx.x; i < (long long)nt * TILE; i += blockDim.x) {
        const int t = (int)(i / TILE), slot = (int)(i % TILE);
        const int4 d = desc[t];
        if (slot == 0 && (d.x < 0 || d.x >= v.S || d.y < 1 || d.y > v.NC || d.z < 0 || d.z > TILE || d.w < 0 || d.w + d.y > next_block)) ++bad;
        if (d.y < 1 || d.y > v.NC || slot >= d.z) continue;
        const int r = rank[i];
        if (r <= PANEL * (d.y - 1) || r > PANEL * d.y) ++bad;
        const int a = aux[i];
        if (side == 0) {
          if (a < 0 || a >= ROPE_LO * ROPE_HI) ++bad;
        } else if (a < 0 || a / TILE >= ntk || kdesc[a / TILE].x != d.x || a % TILE >= kdesc[a / TILE].z) {
          ++bad;
        }
      }
    }
    for (int c = 0; c < v.NC; ++c) {
      const int n = v.kcc(l)[c];
      if (n < 0 || n > v.NT) { if (threadIdx.x == 0) ++bad; continue; }
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int t = v.kct(l)[(size_t)c * v.NT + i];
        if (t < 0 || t >= v.ntiles(l)[0] || v.desc(l, 0)[t].y != c + 1) ++bad;
      }
    }
    for (int s = 0; s < v.S; ++s) {
      const int n = v.svc(l)[s];
      if (n < 0 || n > v.TPS) { if (threadIdx.x == 0) ++bad; continue; }
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int t = v.svt(l)[(size_t)s * v.TPS + i];
        if (t < 0 || t >= v.ntiles(l)[1] || v.desc(l, 1)[t].x != s) ++bad;
      }
    }
  }
  if (bad) atomicAdd(&s_bad, bad);
  __syncthreads();
  if (threadIdx.x == 0) {
    out[0] = s_bad;
    if (s_bad) set_status(v, TWKV_ERR_DEVICE_CHECK);
  }
}

cudaError_t launch_cache_check(const DevView& v, int layer, const unsigned long long* guards_dev, int n_guards, unsigned long long* out_dev,
                               cudaStream_t st) {
  cache_check_kernel<<<1, 1024, 0, st>>>(v, layer < 0 ? 0 : layer, layer < 0 ? v.L : layer + 1, guards_dev, n_guards, out_dev);
  count_launch();
  return cudaGetLastError();
}

}  // namespace twkv
