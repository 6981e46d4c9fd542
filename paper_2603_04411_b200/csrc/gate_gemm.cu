// Gate logits of Eq. 5: Z = X~ W + b for the K side and the V side (COMPUTE mode).
// A dense contraction [n_tok x d_kv] x [d_kv x d_kv]: 128 x 128 output tiles on the tensor cores,
// 16-bit operands, fp32 accumulation, bias added in the epilogue.
#include "twkv_dev.h"
#include "mma_util.cuh"

namespace twkv {

constexpr int GG_STAGES = 3;
constexpr int GG_THREADS = 256;

template <bool BF16>
__global__ void __launch_bounds__(GG_THREADS, 1)
gate_gemm_kernel(const unsigned short* __restrict__ Xk, const unsigned short* __restrict__ Xv,
                 const unsigned short* __restrict__ Wk, const unsigned short* __restrict__ Wv,
                 const float* __restrict__ bk, const float* __restrict__ bv, int n_tok, int d, float* __restrict__ Z) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* sA = smem;
  unsigned char* sB = smem + GG_STAGES * 16384;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int side = blockIdx.z, m0 = blockIdx.x * 128, n0 = blockIdx.y * 128;
  const unsigned short* X = side ? Xv : Xk;
  const unsigned short* W = side ? Wv : Wk;
  const float* bias = side ? bv : bk;
  const int iters = d / 64;
  auto issue = [&](int it) {
    if (it < iters) {
      const int st = it % GG_STAGES;
      const unsigned dA = smem_u32(sA + st * 16384), dB = smem_u32(sB + st * 16384);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = tid + i * GG_THREADS, row = c >> 3, ch = c & 7;
        const int grow = min(m0 + row, n_tok - 1);            // rows past the end repeat the last row (never stored)
        cp_async16(dA + row * 128 + ((ch ^ (row & 7)) << 4),
                   reinterpret_cast<const unsigned char*>(X) + ((size_t)grow * d + it * 64) * 2 + ch * 16);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = tid + i * GG_THREADS, kr = c >> 4, ch = c & 15;
        cp_async16(dB + kr * 256 + ((ch ^ (kr & 7)) << 4),
                   reinterpret_cast<const unsigned char*>(W) + ((size_t)(it * 64 + kr) * d + n0) * 2 + ch * 16);
      }
    }
    cp_async_commit();
  };
  for (int it = 0; it < GG_STAGES - 1; ++it) issue(it);
  float acc[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
  const int mat = lane >> 3, rin = lane & 7;
  for (int it = 0; it < iters; ++it) {
    const int st = it % GG_STAGES;
    cp_async_wait<GG_STAGES - 2>();
    __syncthreads();
    issue(it + GG_STAGES - 1);
    const unsigned aBase = smem_u32(sA + st * 16384), bBase = smem_u32(sB + st * 16384);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      unsigned a[4];
      {
        const int row = warp * 16 + rin + (mat & 1) * 8, kc = ks * 2 + (mat >> 1);
        ldsm_x4(a, aBase + row * 128 + ((kc ^ (row & 7)) << 4));
      }
#pragma unroll
      for (int np = 0; np < 8; ++np) {
        unsigned b[4];
        const int kr = ks * 16 + rin + (mat & 1) * 8, nc = np * 2 + (mat >> 1);
        ldsm_x4_t(b, bBase + kr * 256 + ((nc ^ (kr & 7)) << 4));
        mma16816<BF16>(acc[np * 2], a, b[0], b[1]);
        mma16816<BF16>(acc[np * 2 + 1], a, b[2], b[3]);
      }
    }
  }
  cp_async_wait<0>();
  const int r0 = m0 + warp * 16 + (lane >> 2), r1 = r0 + 8;
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    const int col = n0 + n * 8 + (lane & 3) * 2;
    const float b0 = bias ? bias[col] : 0.f, b1 = bias ? bias[col + 1] : 0.f;
    if (r0 < n_tok) *reinterpret_cast<float2*>(Z + ((size_t)r0 * 2 + side) * d + col) = make_float2(acc[n][0] + b0, acc[n][1] + b1);
    if (r1 < n_tok) *reinterpret_cast<float2*>(Z + ((size_t)r1 * 2 + side) * d + col) = make_float2(acc[n][2] + b0, acc[n][3] + b1);
  }
}

cudaError_t launch_gate_logits(const DevView& v, const LayerParams& lp, const void* K, const void* V, int n_tok,
                               float* logits, cudaStream_t st) {
  if (n_tok <= 0) return cudaSuccess;
  const size_t smem = 2 * GG_STAGES * 16384;
  const dim3 grid((n_tok + 127) / 128, v.d_kv / 128, 2);
  ProfScope ps(TWKV_K_GATE_GEMM, st);
  auto X = [](const void* p) { return reinterpret_cast<const unsigned short*>(p); };
  if (v.dtype == TWKV_BF16) {
    cudaFuncSetAttribute(gate_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    gate_gemm_kernel<true><<<grid, GG_THREADS, smem, st>>>(X(K), X(V), X(lp.W_k), X(lp.W_v), lp.b_k, lp.b_v, n_tok, v.d_kv, logits);
  } else {
    cudaFuncSetAttribute(gate_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    gate_gemm_kernel<false><<<grid, GG_THREADS, smem, st>>>(X(K), X(V), X(lp.W_k), X(lp.W_v), lp.b_k, lp.b_v, n_tok, v.d_kv, logits);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace twkv
