// Soft gating (Eq. 6, Eq. 7) and the soft mask's Retain Rate (the R that Eq. 9 penalises), from gate logits.
//
// Warp per (token, side) row.  Each lane owns d/32 consecutive logits, so the cumulative sum of Eq. 6 is a
// lane-local running sum plus a warp scan of the lane totals, exactly as in the rank kernel:
//   p = softmax(z) (Eq. 5), c_n = sum_{j<=n} p_j, m_i = c_{d+1-i} (Eq. 6, Flip as an index reversal),
//   x^_i = x~_i m_i (Eq. 7),  R = (1/d) sum_i m_i (Eq. 4 applied to the soft mask).
// Outputs are fp32; any of them may be absent.
#include "twkv_dev.h"
#include "mma_util.cuh"

namespace twkv {

template <bool BF16>
__global__ void __launch_bounds__(256) gate_soft_kernel(const float* __restrict__ logits, const unsigned short* __restrict__ Xk,
                                                        const unsigned short* __restrict__ Xv, float* __restrict__ mk,
                                                        float* __restrict__ mv, float* __restrict__ xhk, float* __restrict__ xhv,
                                                        float* __restrict__ retain, int n_rows, int d) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= n_rows) return;
  const int tok = w >> 1, side = w & 1;
  const int per = d >> 5;                       // 4 .. 32, multiple of 4
  const float* z = logits + (size_t)w * d + lane * per;
  float v[32];
  float mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    if (i < per) {
      const float4 t = *reinterpret_cast<const float4*>(z + i);
      v[i] = t.x; v[i + 1] = t.y; v[i + 2] = t.z; v[i + 3] = t.w;
      mx = fmaxf(mx, fmaxf(fmaxf(t.x, t.y), fmaxf(t.z, t.w)));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float run = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    if (i < per) { run += expf(v[i] - mx); v[i] = run; }      // lane-local inclusive sums
  }
  float incl = run;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  const float total = __shfl_sync(0xffffffffu, incl, 31);
  const float offset = incl - run, inv = 1.f / total;
  float* m_out = side ? mv : mk;
  float* xh_out = side ? xhv : xhk;
  const unsigned short* x = (side ? Xv : Xk) + (size_t)tok * d;
  float msum = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    if (i < per) {
      const float c = (offset + v[i]) * inv;                 // c_n, n = lane * per + i (0-based)
      const int at = d - 1 - (lane * per + i);               // Flip: m at index d - 1 - n
      msum += c;
      if (m_out) m_out[(size_t)tok * d + at] = c;
      if (xh_out) xh_out[(size_t)tok * d + at] = to_f32<BF16>(x[at]) * c;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) msum += __shfl_xor_sync(0xffffffffu, msum, o);
  if (lane == 0 && retain) retain[w] = msum / (float)d;
}

cudaError_t launch_gate_soft(const DevView& v, const float* logits, const void* K, const void* V, float* mk, float* mv, float* xhk,
                             float* xhv, float* retain, int n_tok, cudaStream_t st) {
  const int rows = 2 * n_tok;
  if (rows == 0) return cudaSuccess;
  ProfScope ps(TWKV_K_GATE_RANK, st);
  const unsigned short* xk = reinterpret_cast<const unsigned short*>(K);
  const unsigned short* xv = reinterpret_cast<const unsigned short*>(V);
  if (v.dtype == TWKV_BF16) gate_soft_kernel<true><<<(rows + 7) / 8, 256, 0, st>>>(logits, xk, xv, mk, mv, xhk, xhv, retain, rows, v.d_kv);
  else gate_soft_kernel<false><<<(rows + 7) / 8, 256, 0, st>>>(logits, xk, xv, mk, mv, xhk, xhv, retain, rows, v.d_kv);
  count_launch();
  return cudaGetLastError();
}

}  // namespace twkv
