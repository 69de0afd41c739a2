// Elementwise kernels: split-K partial reduction (fixed order, deterministic) with the scale by
// s and the bf16 re-encoding that feeds U = x A^T and V = dY B back to the tensor cores, and the
// fused multi-tensor AdamW step on the LoRA parameters.
#include "common.cuh"

namespace templora {
namespace {

constexpr int kMaxJobs = 32;
struct ReduceBatch {
  int n_jobs;
  int block_start[kMaxJobs + 1];  // first block of each job
  ReduceJob job[kMaxJobs];
};
constexpr int kRedThreads = 256;
constexpr int kRedPerBlock = kRedThreads * 4;

__global__ void __launch_bounds__(kRedThreads) reduce_partials_kernel(const __grid_constant__ ReduceBatch b) {
  pdl_prologue();
  int j = 0;
  while (j + 1 < b.n_jobs && (int)blockIdx.x >= b.block_start[j + 1]) ++j;
  const ReduceJob &jb = b.job[j];
  long long i0 = ((long long)(blockIdx.x - b.block_start[j]) * kRedThreads + threadIdx.x) * 4;
  if (i0 >= jb.n) return;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  const bool vec = (i0 + 4 <= jb.n) && ((jb.stride & 3) == 0) && ((reinterpret_cast<uintptr_t>(jb.part) & 15) == 0);
  for (int k = 0; k < jb.n_parts; ++k) {
    const float *p = jb.part + (long long)k * jb.stride + i0;
    if (vec) {
      float4 t = *reinterpret_cast<const float4 *>(p);
      acc[0] += t.x; acc[1] += t.y; acc[2] += t.z; acc[3] += t.w;
    } else {
      for (int e = 0; e < 4; ++e)
        if (i0 + e < jb.n) acc[e] += p[e];
    }
  }
  for (int e = 0; e < 4; ++e) {
    if (i0 + e >= jb.n) break;
    if (jb.out_f32) {
      float val = jb.scale_f32 * acc[e];
      jb.out_f32[i0 + e] = jb.accumulate_f32 ? jb.out_f32[i0 + e] + val : val;
    }
    if (jb.out_bf16) jb.out_bf16[i0 + e] = __float2bfloat16_rn(jb.scale_bf16 * acc[e]);
  }
}

// ---------------------------------------------------------------- AdamW ----
constexpr int kMaxAdam = 64;
struct AdamTensor {
  float *p, *m, *v;
  const float *g;
  __nv_bfloat16 *work;
  long long n;
};
struct AdamBatch {
  int n_tensors;
  int block_start[kMaxAdam + 1];
  AdamTensor t[kMaxAdam];
  float decay;        // 1 - lr*wd
  float beta1, beta2, omb1, omb2;
  float step_size;    // lr / (1 - beta1^t)
  float inv_sqrt_bc2; // 1 / sqrt(1 - beta2^t)
  float eps;
};
constexpr int kAdamThreads = 256;
constexpr int kAdamPerBlock = kAdamThreads * 4 * 4;  // 4 float4 per thread

__device__ __forceinline__ void adam_one(float &p, float &m, float &v, float g, const AdamBatch &b) {
  p = p * b.decay;
  m = b.beta1 * m + b.omb1 * g;
  v = b.beta2 * v + b.omb2 * g * g;
  float denom = sqrtf(v) * b.inv_sqrt_bc2 + b.eps;
  p = p - b.step_size * (m / denom);
}

__global__ void __launch_bounds__(kAdamThreads) adamw_kernel(const __grid_constant__ AdamBatch b) {
  pdl_prologue();
  int j = 0;
  while (j + 1 < b.n_tensors && (int)blockIdx.x >= b.block_start[j + 1]) ++j;
  const AdamTensor &t = b.t[j];
  const long long base = (long long)(blockIdx.x - b.block_start[j]) * kAdamPerBlock;
  const bool vec = ((reinterpret_cast<uintptr_t>(t.p) | reinterpret_cast<uintptr_t>(t.m) |
                     reinterpret_cast<uintptr_t>(t.v) | reinterpret_cast<uintptr_t>(t.g)) & 15) == 0 &&
                   (t.work == nullptr || (reinterpret_cast<uintptr_t>(t.work) & 7) == 0);
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    long long i0 = base + ((long long)it * kAdamThreads + threadIdx.x) * 4;
    if (i0 >= t.n) break;
    if (vec && i0 + 4 <= t.n) {
      float4 p = *reinterpret_cast<float4 *>(t.p + i0);
      float4 m = *reinterpret_cast<float4 *>(t.m + i0);
      float4 v = *reinterpret_cast<float4 *>(t.v + i0);
      float4 g = __ldg(reinterpret_cast<const float4 *>(t.g + i0));
      adam_one(p.x, m.x, v.x, g.x, b);
      adam_one(p.y, m.y, v.y, g.y, b);
      adam_one(p.z, m.z, v.z, g.z, b);
      adam_one(p.w, m.w, v.w, g.w, b);
      *reinterpret_cast<float4 *>(t.p + i0) = p;
      *reinterpret_cast<float4 *>(t.m + i0) = m;
      *reinterpret_cast<float4 *>(t.v + i0) = v;
      if (t.work) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(p.x, p.y), hi = __floats2bfloat162_rn(p.z, p.w);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t *>(&lo);
        w.y = *reinterpret_cast<uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(t.work + i0) = w;
      }
    } else {
      for (int e = 0; e < 4 && i0 + e < t.n; ++e) {
        float p = t.p[i0 + e], m = t.m[i0 + e], v = t.v[i0 + e];
        adam_one(p, m, v, t.g[i0 + e], b);
        t.p[i0 + e] = p; t.m[i0 + e] = m; t.v[i0 + e] = v;
        if (t.work) t.work[i0 + e] = __float2bfloat16_rn(p);
      }
    }
  }
}

}  // namespace

templora_status_t reduce_partials_batch(const ReduceJob *jobs, int n_jobs, cudaStream_t st) {
  for (int j0 = 0; j0 < n_jobs; j0 += kMaxJobs) {
    ReduceBatch b;
    b.n_jobs = (n_jobs - j0 < kMaxJobs) ? n_jobs - j0 : kMaxJobs;
    int blocks = 0;
    for (int j = 0; j < b.n_jobs; ++j) {
      b.job[j] = jobs[j0 + j];
      if (b.job[j].n <= 0 || b.job[j].n_parts <= 0 || !b.job[j].part) return TEMPLORA_ERR_INVALID_ARG;
      b.block_start[j] = blocks;
      blocks += (int)((b.job[j].n + kRedPerBlock - 1) / kRedPerBlock);
    }
    b.block_start[b.n_jobs] = blocks;
    {
      LaunchScope scope(kKindReduce, st);
      TL_CUDA_CHECK(launch_pdl(reduce_partials_kernel, dim3(blocks), dim3(kRedThreads), 0, st, b));
    }
    TL_CUDA_CHECK(cudaGetLastError());
  }
  return TEMPLORA_OK;
}

templora_status_t adamw_launch(const templora_param_t *params, int n_params, float lr, float beta1, float beta2,
                               float eps, float wd, int64_t step, int work_bf16, cudaStream_t st) {
  // constants in double, rounded once to fp32 (1 - beta2 formed in fp32 would be off by 5e-5 relative)
  const double bc1 = 1.0 - pow((double)beta1, (double)step);
  const double bc2 = 1.0 - pow((double)beta2, (double)step);
  for (int t0 = 0; t0 < n_params; t0 += kMaxAdam) {
    AdamBatch b;
    b.n_tensors = (n_params - t0 < kMaxAdam) ? n_params - t0 : kMaxAdam;
    b.decay = (float)(1.0 - (double)lr * (double)wd);
    b.beta1 = beta1; b.beta2 = beta2;
    b.omb1 = (float)(1.0 - (double)beta1);
    b.omb2 = (float)(1.0 - (double)beta2);
    b.step_size = (float)((double)lr / bc1);
    b.inv_sqrt_bc2 = (float)(1.0 / sqrt(bc2));
    b.eps = eps;
    long long blocks = 0;
    for (int i = 0; i < b.n_tensors; ++i) {
      const templora_param_t &p = params[t0 + i];
      b.t[i] = AdamTensor{p.master, p.m, p.v, p.grad, work_bf16 ? reinterpret_cast<__nv_bfloat16 *>(p.work) : nullptr,
                          (long long)p.n};
      b.block_start[i] = (int)blocks;
      blocks += (p.n + kAdamPerBlock - 1) / kAdamPerBlock;
    }
    if (blocks > 0x7fffffffLL) return TEMPLORA_ERR_UNSUPPORTED;
    b.block_start[b.n_tensors] = (int)blocks;
    {
      LaunchScope scope(kKindAdamW, st);
      TL_CUDA_CHECK(launch_pdl(adamw_kernel, dim3((unsigned)blocks), dim3(kAdamThreads), 0, st, b));
    }
    TL_CUDA_CHECK(cudaGetLastError());
  }
  return TEMPLORA_OK;
}

}  // namespace templora
