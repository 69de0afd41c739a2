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
  if (vec) {
    // four slabs' loads are issued before any is added (the sum still runs in slab order): one memory round trip
    // per four slabs instead of one per slab
    int k = 0;
    for (; k + 4 <= jb.n_parts; k += 4) {
      const float *p = jb.part + (long long)k * jb.stride + i0;
      const float4 t0 = *reinterpret_cast<const float4 *>(p), t1 = *reinterpret_cast<const float4 *>(p + jb.stride),
                   t2 = *reinterpret_cast<const float4 *>(p + 2 * jb.stride), t3 = *reinterpret_cast<const float4 *>(p + 3 * jb.stride);
      acc[0] += t0.x; acc[1] += t0.y; acc[2] += t0.z; acc[3] += t0.w;
      acc[0] += t1.x; acc[1] += t1.y; acc[2] += t1.z; acc[3] += t1.w;
      acc[0] += t2.x; acc[1] += t2.y; acc[2] += t2.z; acc[3] += t2.w;
      acc[0] += t3.x; acc[1] += t3.y; acc[2] += t3.z; acc[3] += t3.w;
    }
    for (; k < jb.n_parts; ++k) {
      const float4 t = *reinterpret_cast<const float4 *>(jb.part + (long long)k * jb.stride + i0);
      acc[0] += t.x; acc[1] += t.y; acc[2] += t.z; acc[3] += t.w;
    }
  } else {
    for (int k = 0; k < jb.n_parts; ++k) {
      const float *p = jb.part + (long long)k * jb.stride + i0;
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

// ---------------------------------------------------------------- dropout ----
// Philox4x32-10 (Salmon et al., SC'11), written from its published definition: ten rounds of
//   (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))
// with the key bumped by the Weyl constants after every round.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

constexpr int kMaxDropJobs = 8;
struct DropoutBatch {
  int n_jobs;
  int block_start[kMaxDropJobs + 1];
  DropoutJob job[kMaxDropJobs];
  uint32_t threshold[kMaxDropJobs];   // dropped iff draw < threshold
  float inv_keep[kMaxDropJobs];       // 1 / (1 - p)
};
constexpr int kDropThreads = 256;

// One thread per group of 8 consecutive elements of a row: writes 8 values of xd and one mask byte.
__global__ void __launch_bounds__(kDropThreads) dropout_apply_kernel(const __grid_constant__ DropoutBatch b) {
  pdl_prologue();
  int j = 0;
  while (j + 1 < b.n_jobs && (int)blockIdx.x >= b.block_start[j + 1]) ++j;
  const DropoutJob &jb = b.job[j];
  const long long groups_per_row = (jb.d_in + 7) / 8;
  const long long gidx = (long long)(blockIdx.x - b.block_start[j]) * kDropThreads + threadIdx.x;
  if (gidx >= jb.T * groups_per_row) return;
  const long long t = gidx / groups_per_row, k0 = (gidx - t * groups_per_row) * 8;
  const uint2 key = make_uint2((uint32_t)jb.seed, (uint32_t)(jb.seed >> 32));
  const uint32_t thr = b.threshold[j];
  const float inv = b.inv_keep[j];
  const uint32_t off_lo = (uint32_t)jb.offset, off_hi = (uint32_t)(jb.offset >> 32);
  const long long idx0 = t * jb.d_in + k0;
  if ((jb.d_in & 7) == 0) {
    // fast path: the 8 elements are two whole Philox blocks and one 16-byte (bf16) or 32-byte (fp32) vector
    const unsigned long long q = (unsigned long long)idx0 >> 2;
    const uint4 d0 = philox4x32_10(make_uint4((uint32_t)q, (uint32_t)(q >> 32), off_lo, off_hi), key);
    const uint4 d1 = philox4x32_10(make_uint4((uint32_t)(q + 1), (uint32_t)((q + 1) >> 32), off_lo, off_hi), key);
    const uint32_t w[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
    uint32_t bits = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) bits |= (w[i] >= thr ? 1u : 0u) << i;
    jb.mask[t * jb.mask_pitch + (k0 >> 3)] = (uint8_t)bits;
    if (jb.dt == TEMPLORA_BF16) {
      uint4 v = *reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(jb.x) + idx0);
      __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(h[e]);
        h[e] = __floats2bfloat162_rn((bits >> (2 * e)) & 1 ? f.x * inv : 0.f, (bits >> (2 * e + 1)) & 1 ? f.y * inv : 0.f);
      }
      *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(jb.xd) + idx0) = v;
    } else {
      const float4 *src = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(jb.x) + idx0);
      float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(jb.xd) + idx0);
      float4 a = src[0], c = src[1];
      a.x = bits & 1 ? a.x * inv : 0.f;  a.y = bits & 2 ? a.y * inv : 0.f;
      a.z = bits & 4 ? a.z * inv : 0.f;  a.w = bits & 8 ? a.w * inv : 0.f;
      c.x = bits & 16 ? c.x * inv : 0.f; c.y = bits & 32 ? c.y * inv : 0.f;
      c.z = bits & 64 ? c.z * inv : 0.f; c.w = bits & 128 ? c.w * inv : 0.f;
      dst[0] = a; dst[1] = c;
    }
    return;
  }
  // general path: any d_in, element by element
  unsigned long long cached_q = ~0ull;
  uint4 draw = make_uint4(0, 0, 0, 0);
  uint32_t bits = 0;
  for (int i = 0; i < 8; ++i) {
    const long long k = k0 + i;
    if (k >= jb.d_in) break;
    const unsigned long long e = (unsigned long long)(idx0 + i), q = e >> 2;
    if (q != cached_q) {
      draw = philox4x32_10(make_uint4((uint32_t)q, (uint32_t)(q >> 32), off_lo, off_hi), key);
      cached_q = q;
    }
    const uint32_t w = (e & 3) == 0 ? draw.x : (e & 3) == 1 ? draw.y : (e & 3) == 2 ? draw.z : draw.w;
    const bool keep = w >= thr;
    if (keep) bits |= 1u << i;
    if (jb.dt == TEMPLORA_BF16) {
      const float xv = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(jb.x)[idx0 + i]);
      reinterpret_cast<__nv_bfloat16 *>(jb.xd)[idx0 + i] = __float2bfloat16_rn(keep ? xv * inv : 0.f);
    } else {
      const float xv = reinterpret_cast<const float *>(jb.x)[idx0 + i];
      reinterpret_cast<float *>(jb.xd)[idx0 + i] = keep ? xv * inv : 0.f;
    }
  }
  jb.mask[t * jb.mask_pitch + (k0 >> 3)] = (uint8_t)bits;
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

templora_status_t dropout_apply_batch(const DropoutJob *jobs, int n_jobs, cudaStream_t st) {
  for (int j0 = 0; j0 < n_jobs; j0 += kMaxDropJobs) {
    DropoutBatch b;
    b.n_jobs = (n_jobs - j0 < kMaxDropJobs) ? n_jobs - j0 : kMaxDropJobs;
    long long blocks = 0;
    for (int j = 0; j < b.n_jobs; ++j) {
      const DropoutJob &jb = jobs[j0 + j];
      if (!jb.x || !jb.xd || !jb.mask || jb.T <= 0 || jb.d_in <= 0 || !(jb.p > 0.f && jb.p < 1.f)) return TEMPLORA_ERR_INVALID_ARG;
      b.job[j] = jb;
      double thr = floor((double)jb.p * 4294967296.0);
      b.threshold[j] = thr >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)thr;
      b.inv_keep[j] = (float)(1.0 / (1.0 - (double)jb.p));
      b.block_start[j] = (int)blocks;
      blocks += (jb.T * ((jb.d_in + 7) / 8) + kDropThreads - 1) / kDropThreads;
    }
    if (blocks > 0x7fffffffLL) return TEMPLORA_ERR_UNSUPPORTED;
    b.block_start[b.n_jobs] = (int)blocks;
    {
      LaunchScope scope(kKindDropout, st);
      TL_CUDA_CHECK(launch_pdl(dropout_apply_kernel, dim3((unsigned)blocks), dim3(kDropThreads), 0, st, b));
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
