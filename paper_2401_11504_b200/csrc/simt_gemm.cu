// Generic-shape GEMM on the plain FP32 pipes:
//     D = alpha1 * A1 B1 + alpha2 * A2 B2 (+ D)
// Operands are addressed through element strides and may be fp32 or bf16, so the one kernel
// serves every product of the LoRA-augmented projection (x W0^T with the s U B^T term fused as
// the second product, dY W0 with s V A, the token-dimension reductions dB = s dY^T U and
// dA = s V^T x) on the fp32 path and for shapes the tensor-core path does not take.
// Accumulation is fp32 in a fixed order (k ascending), so results are run-to-run identical.
#include "common.cuh"

namespace templora {
namespace {

constexpr int TM = 64, TN = 64, TK = 16, NT = 256;

__device__ __forceinline__ float load_el(const Operand &o, long long i, long long k) {
  long long idx = i * o.s0 + k * o.s1;
  if (o.dt == TEMPLORA_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(o.p)[idx]);
  return reinterpret_cast<const float *>(o.p)[idx];
}

__device__ __forceinline__ void product(const Operand &A, const Operand &B, int M, int N, int K, int m0, int n0,
                                        float (&acc)[4][4], float (*sA)[TM + 1], float (*sB)[TN + 1]) {
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  for (int k0 = 0; k0 < K; k0 += TK) {
    // stage a TM x TK slab of A and a TK x TN slab of B (zero outside the matrix)
    for (int e = tid; e < TM * TK; e += NT) {
      int kk, ii;
      if (A.s1 == 1) { kk = e % TK; ii = e / TK; } else { ii = e % TM; kk = e / TM; }
      int gi = m0 + ii, gk = k0 + kk;
      sA[kk][ii] = (gi < M && gk < K) ? load_el(A, gi, gk) : 0.f;
    }
    for (int e = tid; e < TN * TK; e += NT) {
      int kk, jj;
      if (B.s0 == 1) { kk = e % TK; jj = e / TK; } else { jj = e % TN; kk = e / TN; }
      int gj = n0 + jj, gk = k0 + kk;
      sB[kk][jj] = (gj < N && gk < K) ? load_el(B, gk, gj) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = sA[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = sB[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(NT) simt_gemm_kernel(const SimtGemm g) {
  __shared__ float sA[TK][TM + 1];
  __shared__ float sB[TK][TN + 1];
  pdl_prologue();
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;

  float acc1[4][4] = {};
  product(g.A1, g.B1, g.M, g.N, g.K1, m0, n0, acc1, sA, sB);
  float acc2[4][4] = {};
  if (g.K2 > 0) product(g.A2, g.B2, g.M, g.N, g.K2, m0, n0, acc2, sA, sB);

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gi = m0 + ty * 4 + i;
    if (gi >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gj = n0 + tx * 4 + j;
      if (gj >= g.N) continue;
      float val = g.alpha1 * acc1[i][j] + g.alpha2 * acc2[i][j];
      if (g.mask && !((g.mask[(long long)gi * g.mask_pitch + (gj >> 3)] >> (gj & 7)) & 1)) val = 0.f;
      long long idx = (long long)gi * g.ds0 + (long long)gj * g.ds1;
      if (g.d_dt == TEMPLORA_BF16) {
        __nv_bfloat16 *d = reinterpret_cast<__nv_bfloat16 *>(g.D);
        d[idx] = __float2bfloat16_rn(g.accumulate ? __bfloat162float(d[idx]) + val : val);
      } else {
        float *d = reinterpret_cast<float *>(g.D);
        d[idx] = g.accumulate ? d[idx] + val : val;
      }
    }
  }
}

}  // namespace

templora_status_t simt_gemm(const SimtGemm &g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.K1 <= 0) return TEMPLORA_ERR_INVALID_ARG;
  dim3 grid((g.N + TN - 1) / TN, (g.M + TM - 1) / TM);
  if (grid.y > 65535u) return TEMPLORA_ERR_UNSUPPORTED;
  {
    LaunchScope scope(kKindSimt, st);
    TL_CUDA_CHECK(launch_pdl(simt_gemm_kernel, grid, dim3(NT), 0, st, g));
  }
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

}  // namespace templora
