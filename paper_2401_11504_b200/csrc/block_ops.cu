// The element-wise steps either side of the projections inside a decoder block's update: the MLP's
// SiLU gating and RMSNorm, forward and backward.  All four are bound by HBM bandwidth: every element is
// read once and written once, 16 bytes per thread per access, arithmetic in fp32.
#include "common.cuh"

namespace templora {
namespace {

constexpr int kThreadsEw = 256;

template <typename T> struct Vec;   // 16 bytes of T
template <> struct Vec<__nv_bfloat16> {
  static constexpr int kN = 8;
  uint4 raw;
  __device__ __forceinline__ void unpack(float (&f)[8]) const {
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 t = __bfloat1622float2(h[i]);
      f[2 * i] = t.x; f[2 * i + 1] = t.y;
    }
  }
  __device__ __forceinline__ void pack(const float (&f)[8]) {
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  }
};
template <> struct Vec<float> {
  static constexpr int kN = 4;
  float4 raw;
  __device__ __forceinline__ void unpack(float (&f)[4]) const { f[0] = raw.x; f[1] = raw.y; f[2] = raw.z; f[3] = raw.w; }
  __device__ __forceinline__ void pack(const float (&f)[4]) { raw = make_float4(f[0], f[1], f[2], f[3]); }
};
__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f(float &o, float v) { o = v; }
__device__ __forceinline__ void from_f(__nv_bfloat16 &o, float v) { o = __float2bfloat16_rn(v); }

// ex2.approx and rcp.approx: about 2 ulp each, far inside the fp32 tolerance; the accurate expf and division
// made the forward gating kernel instruction-bound (0.70 of the copy bandwidth)
__device__ __forceinline__ float sigmoidf_(float g) { return __fdividef(1.f, 1.f + __expf(-g)); }

// ---------------------------------------------------------------- SiLU gating
// h = SiLU(gate) * up over n elements; BWD: dgate = dh * up * SiLU'(gate), dup = dh * SiLU(gate).
template <typename T, bool BWD>
__global__ void __launch_bounds__(kThreadsEw) swiglu_kernel(const T *__restrict__ gate, const T *__restrict__ up,
                                                            const T *__restrict__ dh, T *__restrict__ out0,
                                                            T *__restrict__ out1, long long n) {
  pdl_prologue();
  constexpr int N = Vec<T>::kN;
  const long long nvec = n / N;
  const long long stride = (long long)gridDim.x * blockDim.x;
  // A CTA takes contiguous chunks of UNR * blockDim vectors (16 KB per tensor at a time: few DRAM pages open at
  // once); a thread has UNR vectors per tensor in flight, all loads of a chunk issued before any is used.
  constexpr int UNR = 4;
  const long long chunk = (long long)UNR * blockDim.x;
  for (long long v0 = (long long)blockIdx.x * chunk + threadIdx.x; v0 - threadIdx.x < nvec; v0 += (long long)gridDim.x * chunk) {
    Vec<T> a[UNR], b[UNR], c[UNR];
#pragma unroll
    for (int k = 0; k < UNR; ++k) {
      const long long v = v0 + (long long)k * blockDim.x;
      if (v < nvec) {
        a[k].raw = reinterpret_cast<const decltype(a[k].raw) *>(gate)[v];
        b[k].raw = reinterpret_cast<const decltype(b[k].raw) *>(up)[v];
        if (BWD) c[k].raw = reinterpret_cast<const decltype(c[k].raw) *>(dh)[v];
      }
    }
#pragma unroll
    for (int k = 0; k < UNR; ++k) {
      const long long v = v0 + (long long)k * blockDim.x;
      if (v >= nvec) break;
      float g[N], u[N], d[N], o0[N], o1[N];
      a[k].unpack(g); b[k].unpack(u);
      if (BWD) c[k].unpack(d);
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const float sg = sigmoidf_(g[i]);
        if (BWD) {
          o0[i] = d[i] * u[i] * sg * (1.f + g[i] * (1.f - sg));
          o1[i] = d[i] * g[i] * sg;
        } else {
          o0[i] = g[i] * sg * u[i];
        }
      }
      Vec<T> r0, r1;
      r0.pack(o0);
      reinterpret_cast<decltype(r0.raw) *>(out0)[v] = r0.raw;
      if (BWD) {
        r1.pack(o1);
        reinterpret_cast<decltype(r1.raw) *>(out1)[v] = r1.raw;
      }
    }
  }
  // ragged tail (n not a multiple of the vector width)
  for (long long e = nvec * N + (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += stride) {
    const float g = to_f(gate[e]), u = to_f(up[e]), sg = sigmoidf_(g);
    if (BWD) {
      const float d = to_f(dh[e]);
      from_f(out0[e], d * u * sg * (1.f + g * (1.f - sg)));
      from_f(out1[e], d * g * sg);
    } else {
      from_f(out0[e], g * sg * u);
    }
  }
}

// ---------------------------------------------------------------- RMSNorm
// One warp per row: a first pass over the row forms the sums (shuffle reduction, no block barrier), a
// second pass reads the row again (from L2, where the first pass has just put it) and writes the result.
// Nothing is staged, so 64 rows per SM are in flight and DRAM sees every byte once.
constexpr int kRowsPerCta = kThreadsEw / 32;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;   // every lane holds the same sum, formed in the same order
}

// FWD: y = x * rstd * w, rstd = 1 / sqrt(mean(x^2) + eps).
// BWD: dx = rstd * (w * dy) - x * rstd^3 / d * sum_j(x_j * w_j * dy_j).
template <typename T, bool BWD>
__global__ void __launch_bounds__(kThreadsEw) rmsnorm_kernel(const T *__restrict__ x, const T *__restrict__ w,
                                                            const T *__restrict__ dy, T *__restrict__ out, int T_rows,
                                                            int d, float eps) {
  pdl_prologue();
  constexpr int N = Vec<T>::kN;
  constexpr int UNR = 4;
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);
  if (row >= T_rows) return;
  const T *xr = x + row * d;
  const T *dr = BWD ? dy + row * d : nullptr;
  T *orow = out + row * d;
  const bool vec = (d % N == 0);   // rows then start on 16-byte boundaries (the base pointers are checked by the host)
  const int nvec = d / N;
  float ss = 0.f, s2 = 0.f;
  if (vec) {
    for (int v0 = lane; v0 - lane < nvec; v0 += 32 * UNR) {
      Vec<T> a[UNR], b[UNR], c[UNR];
#pragma unroll
      for (int k = 0; k < UNR; ++k) {
        const int v = v0 + 32 * k;
        if (v < nvec) {
          a[k].raw = reinterpret_cast<const decltype(a[k].raw) *>(xr)[v];
          if (BWD) {
            b[k].raw = reinterpret_cast<const decltype(b[k].raw) *>(dr)[v];
            c[k].raw = reinterpret_cast<const decltype(c[k].raw) *>(w)[v];
          }
        }
      }
#pragma unroll
      for (int k = 0; k < UNR; ++k) {
        if (v0 + 32 * k >= nvec) break;
        float fx[N];
        a[k].unpack(fx);
#pragma unroll
        for (int i = 0; i < N; ++i) ss += fx[i] * fx[i];
        if (BWD) {
          float fd[N], fw[N];
          b[k].unpack(fd); c[k].unpack(fw);
#pragma unroll
          for (int i = 0; i < N; ++i) s2 += fx[i] * fw[i] * fd[i];
        }
      }
    }
  } else {
    for (int j = lane; j < d; j += 32) {
      const float fx = to_f(xr[j]);
      ss += fx * fx;
      if (BWD) s2 += fx * to_f(w[j]) * to_f(dr[j]);
    }
  }
  ss = warp_sum(ss);
  if (BWD) s2 = warp_sum(s2);
  const float rstd = rsqrtf(ss / (float)d + eps);
  const float coef = BWD ? rstd * rstd * rstd * s2 / (float)d : 0.f;
  if (vec) {
    for (int v0 = lane; v0 - lane < nvec; v0 += 32 * UNR) {
      Vec<T> a[UNR], b[UNR], c[UNR];
#pragma unroll
      for (int k = 0; k < UNR; ++k) {
        const int v = v0 + 32 * k;
        if (v < nvec) {
          a[k].raw = reinterpret_cast<const decltype(a[k].raw) *>(xr)[v];
          c[k].raw = reinterpret_cast<const decltype(c[k].raw) *>(w)[v];
          if (BWD) b[k].raw = reinterpret_cast<const decltype(b[k].raw) *>(dr)[v];
        }
      }
#pragma unroll
      for (int k = 0; k < UNR; ++k) {
        const int v = v0 + 32 * k;
        if (v >= nvec) break;
        float fx[N], fw[N], fd[N], o[N];
        a[k].unpack(fx); c[k].unpack(fw);
        if (BWD) b[k].unpack(fd);
#pragma unroll
        for (int i = 0; i < N; ++i) o[i] = BWD ? rstd * fw[i] * fd[i] - fx[i] * coef : fx[i] * rstd * fw[i];
        Vec<T> r;
        r.pack(o);
        reinterpret_cast<decltype(r.raw) *>(orow)[v] = r.raw;
      }
    }
  } else {
    for (int j = lane; j < d; j += 32) {
      const float fx = to_f(xr[j]), fw = to_f(w[j]);
      from_f(orow[j], BWD ? rstd * fw * to_f(dr[j]) - fx * coef : fx * rstd * fw);
    }
  }
}

int ew_grid(long long nvec) {
  long long g = (nvec + kThreadsEw - 1) / kThreadsEw;
  const long long cap = 148LL * 8;   // a few resident CTAs per SM; the loop strides over the rest
  if (g > cap) g = cap;
  return g < 1 ? 1 : (int)g;
}

template <typename T>
templora_status_t swiglu_launch(bool bwd, const void *gate, const void *up, const void *dh, void *o0, void *o1,
                                long long n, cudaStream_t st) {
  const int grid = ew_grid(n / Vec<T>::kN / 4);   // a CTA's thread handles four vectors per chunk
  LaunchScope scope(kKindBlockOps, st);
  if (bwd)
    TL_CUDA_CHECK(launch_pdl(swiglu_kernel<T, true>, dim3(grid), dim3(kThreadsEw), 0, st, (const T *)gate, (const T *)up,
                             (const T *)dh, (T *)o0, (T *)o1, n));
  else
    TL_CUDA_CHECK(launch_pdl(swiglu_kernel<T, false>, dim3(grid), dim3(kThreadsEw), 0, st, (const T *)gate,
                             (const T *)up, (const T *)nullptr, (T *)o0, (T *)nullptr, n));
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

template <typename T>
templora_status_t rmsnorm_launch(bool bwd, const void *x, const void *w, const void *dy, void *out, int T_rows, int d,
                                 float eps, cudaStream_t st) {
  const int grid = (T_rows + kRowsPerCta - 1) / kRowsPerCta;
  LaunchScope scope(kKindBlockOps, st);
  if (bwd)
    TL_CUDA_CHECK(launch_pdl(rmsnorm_kernel<T, true>, dim3(grid), dim3(kThreadsEw), 0, st, (const T *)x, (const T *)w,
                             (const T *)dy, (T *)out, T_rows, d, eps));
  else
    TL_CUDA_CHECK(launch_pdl(rmsnorm_kernel<T, false>, dim3(grid), dim3(kThreadsEw), 0, st, (const T *)x, (const T *)w,
                             (const T *)nullptr, (T *)out, T_rows, d, eps));
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

bool aligned16p(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace templora

using namespace templora;

extern "C" {

templora_status_t templora_swiglu_fwd(int64_t n, int32_t dtype, const void *gate, const void *up, void *h, void *stream) {
  if (n <= 0 || !gate || !up || !h) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16p(gate) || !aligned16p(up) || !aligned16p(h)) return TEMPLORA_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (dtype == TEMPLORA_BF16) return swiglu_launch<__nv_bfloat16>(false, gate, up, nullptr, h, nullptr, n, st);
  if (dtype == TEMPLORA_F32) return swiglu_launch<float>(false, gate, up, nullptr, h, nullptr, n, st);
  return TEMPLORA_ERR_UNSUPPORTED;
}

templora_status_t templora_swiglu_bwd(int64_t n, int32_t dtype, const void *gate, const void *up, const void *dh,
                                      void *dgate, void *dup, void *stream) {
  if (n <= 0 || !gate || !up || !dh || !dgate || !dup) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16p(gate) || !aligned16p(up) || !aligned16p(dh) || !aligned16p(dgate) || !aligned16p(dup))
    return TEMPLORA_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (dtype == TEMPLORA_BF16) return swiglu_launch<__nv_bfloat16>(true, gate, up, dh, dgate, dup, n, st);
  if (dtype == TEMPLORA_F32) return swiglu_launch<float>(true, gate, up, dh, dgate, dup, n, st);
  return TEMPLORA_ERR_UNSUPPORTED;
}

templora_status_t templora_rmsnorm_fwd(int32_t T, int32_t d, int32_t dtype, const void *x, const void *w, float eps,
                                       void *y, void *stream) {
  if (T <= 0 || d <= 0 || !x || !w || !y || !(eps >= 0.f)) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16p(x) || !aligned16p(w) || !aligned16p(y)) return TEMPLORA_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (dtype == TEMPLORA_BF16) return rmsnorm_launch<__nv_bfloat16>(false, x, w, nullptr, y, T, d, eps, st);
  if (dtype == TEMPLORA_F32) return rmsnorm_launch<float>(false, x, w, nullptr, y, T, d, eps, st);
  return TEMPLORA_ERR_UNSUPPORTED;
}

templora_status_t templora_rmsnorm_bwd(int32_t T, int32_t d, int32_t dtype, const void *x, const void *w, const void *dy,
                                       float eps, void *dx, void *stream) {
  if (T <= 0 || d <= 0 || !x || !w || !dy || !dx || !(eps >= 0.f)) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16p(x) || !aligned16p(w) || !aligned16p(dy) || !aligned16p(dx)) return TEMPLORA_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (dtype == TEMPLORA_BF16) return rmsnorm_launch<__nv_bfloat16>(true, x, w, dy, dx, T, d, eps, st);
  if (dtype == TEMPLORA_F32) return rmsnorm_launch<float>(true, x, w, dy, dx, T, d, eps, st);
  return TEMPLORA_ERR_UNSUPPORTED;
}

}  // extern "C"
