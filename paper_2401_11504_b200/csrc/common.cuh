// Shared declarations of the Temp-Lora CUDA library (internal; the public ABI is include/templora.h).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <utility>

#include "templora.h"

namespace templora {

// ---- device status record at the head of every workspace -------------------
// code: templora_status_t (0 = ok); where: location tag of the first failure.
struct DeviceStatus {
  int32_t code;
  int32_t where;
  int32_t sched_next;   // tensor-core kernel: next work item to hand out (zero between launches)
  int32_t sched_done;   // tensor-core kernel: CTAs that have finished (zero between launches)
  int32_t pad[60];
};
static_assert(sizeof(DeviceStatus) == 256, "status record is 256 bytes");

constexpr size_t kWsAlign = 1024;
constexpr size_t kStatusBytes = 1024;  // status record + padding; scratch starts here

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

#define TL_CUDA_CHECK(expr)                                   \
  do {                                                        \
    cudaError_t _e = (expr);                                  \
    if (_e != cudaSuccess) return TEMPLORA_ERR_CUDA;          \
  } while (0)

#define TL_TRY(expr)                                          \
  do {                                                        \
    templora_status_t _s = (expr);                            \
    if (_s != TEMPLORA_OK) return _s;                         \
  } while (0)

// ---- launch accounting (timing.cu) -------------------------------------------
enum KernelKind {
  kKindTcMain = 0,     // tensor-core GEMM, 256-wide tiles: y and dX with the rank-r term fused
  kKindTcSkinny = 1,   // tensor-core GEMM, 64-wide tiles: U, V, dB, dA
  kKindTcDecode = 2,   // tensor-core GEMM, 16-wide tiles: decode-time W0 stream
  kKindReduce = 3,     // split-K partial reduction / bf16 re-encoding
  kKindAdamW = 4,
  kKindSimt = 5,       // generic-shape GEMM
  kKindDecodeFinish = 6,
  kKindDropout = 7,        // dropout mask + masked copy of x
  kKindTcDropoutTerm = 8,  // tensor-core second pass adding the masked rank-r term to dX
  kKindBlockOps = 9,       // SiLU gating and RMSNorm, forward and backward
  kKindCount = 10
};
// Construct right before a kernel launch and destroy right after it.
class LaunchScope {
 public:
  LaunchScope(int kind, cudaStream_t st);
  ~LaunchScope();
  LaunchScope(const LaunchScope &) = delete;
  LaunchScope &operator=(const LaunchScope &) = delete;
 private:
  int kind_;
  cudaStream_t st_;
  cudaEvent_t a_, b_;
};

// ---- programmatic dependent launch ----------------------------------------------
// Every kernel of the library starts with pdl_prologue(): it waits until the kernels before it on
// the stream have completed and flushed (so ordering is exactly that of plain stream launches)
// and then lets the kernel after it be scheduled early, which hides that kernel's launch latency
// behind this one's execution.  launch_pdl() launches with that attribute set.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif

// ---- generic (SIMT) GEMM:  D = alpha1 * A1 B1 + alpha2 * A2 B2 (+ D) --------
// Element (i,k) of an operand lives at p[i*s0 + k*s1]; dt is a templora_dtype_t.
struct Operand {
  const void *p;
  int32_t dt;
  long long s0, s1;
};
struct SimtGemm {
  int M, N, K1, K2;          // K2 = 0: no second product
  Operand A1, B1, A2, B2;    // A(i,k), B(k,j)
  float alpha1, alpha2;
  void *D;
  int32_t d_dt;
  long long ds0, ds1;
  int accumulate;            // add to the existing contents of D
  const uint8_t *mask;       // optional keep bits over D's (i, j): masked-out elements add nothing
  long long mask_pitch;
};
templora_status_t simt_gemm(const SimtGemm &g, cudaStream_t st);

// ---- elementwise helpers ----------------------------------------------------
// One reduction of split-K partial slabs, summed in slab order (deterministic):
//   acc[i]      = sum_k part[k*stride + i]
//   out_f32[i]  = scale_f32  * acc[i]  (+ previous contents when accumulate_f32)   if out_f32
//   out_bf16[i] = bf16(scale_bf16 * acc[i])                                        if out_bf16
struct ReduceJob {
  const float *part;
  int n_parts;
  long long stride, n;
  float scale_bf16;
  float scale_f32;
  float *out_f32;
  int accumulate_f32;
  __nv_bfloat16 *out_bf16;
};
templora_status_t reduce_partials_batch(const ReduceJob *jobs, int n_jobs, cudaStream_t st);

// ---- LoRA dropout -----------------------------------------------------------------
// xd = x * keep / (1 - p) in the storage type of x, and the keep mask as bits: byte j of row t
// holds elements 8j .. 8j+7 (bit i = element 8j+i), mask_pitch bytes per row.
struct DropoutJob {
  const void *x;
  void *xd;
  uint8_t *mask;
  long long T, d_in, mask_pitch;
  int32_t dt;
  float p;
  uint64_t seed, offset;
};
templora_status_t dropout_apply_batch(const DropoutJob *jobs, int n_jobs, cudaStream_t st);
inline long long dropout_mask_pitch(long long d_in) { return ((d_in + 7) / 8 + 15) / 16 * 16; }

// ---- AdamW --------------------------------------------------------------------
templora_status_t adamw_launch(const templora_param_t *params, int n_params, float lr, float beta1, float beta2,
                               float eps, float wd, int64_t step, int work_bf16, cudaStream_t st);

// ---- tensor-core (tcgen05) grouped GEMM ---------------------------------------
// D[M,N] = Aop[M,K] Bop[N,K]^T  (+ Aext[M,Kext] Bext[N,Kext]^T), bf16 operands, fp32 accumulation.
// *_mn = 0: operand stored with K contiguous (rows = M or N, pitch ld elements)
// *_mn = 1: operand stored with M (or N) contiguous (rows = K, pitch ld elements)
struct TcProblem {
  int M, N, K, Kext;
  const void *A, *B, *Aext, *Bext;
  long long lda, ldb, ldaext, ldbext;
  int a_mn, b_mn;
  int splits;                 // split-K factor (>= 1); split i writes out + i*out_split
  void *out;
  int out_f32;                // 1: fp32 output, 0: bf16
  long long out_s0, out_s1;   // element (i,j) of D goes to out[i*out_s0 + j*out_s1]
  long long out_split;        // element stride between split-K partial outputs
  // optional epilogue "add under a mask": out = out_old + keep(i, j) ? epi_scale * D(i, j) : 0
  // (keep bits as written by dropout_apply_batch; out must be row-major, out_s1 == 1)
  const uint8_t *epi_mask;
  long long epi_mask_pitch;
  float epi_scale;
  // further operand pairs accumulated into the same output (input gradients of projections that share
  // their input, summed): D += Ax[e][M, Kx[e]] Bx[e][N, Kx[e]]^T, stored like A and B (same a_mn, b_mn);
  // not with split-K
  int n_extra;
  const void *Ax[4], *Bx[4];
  long long ldax[4], ldbx[4];
  int Kx[4];
  // CTA-pair kernel only: the MLP's gating fused into the epilogue.
  //   epi_mode 1, "gate | up" forward: one problem computes both projections of the same input.  A (and Aext =
  //     s*U_gate, Aext1 = s*U_up) as usual; B, Bext describe the gate projection (W_gate [N, K], B_gate [N, Kext]),
  //     B1, Bext1 the up projection; N = d_ff.  Outputs, all [M, N] bf16 row-major with pitch out_s0:
  //     out = gate, out1 = up (the pre-activations, kept for the backward), out2 = h = SiLU(gate) * up.
  //   epi_mode 2, input gradient of the down projection with the gating's backward: D = dh is not stored;
  //     out = dgate = dh * up * SiLU'(gate), out1 = dup = dh * SiLU(gate), read from epi_in0 = gate, epi_in1 = up
  //     ([M, N] bf16, pitch out_s0).
  int epi_mode;
  const void *B1, *Bext1, *Aext1;
  long long ldb1, ldbext1, ldaext1;
  void *out1, *out2;
  const void *epi_in0, *epi_in1;
  // tc_decode_cluster only: role 0 = y of a projection, 1 = its u = A x^T (stored as bf16(epi_scale * u));
  // flag = the projection's index within the launch
  int role, flag;
};
constexpr int kTcMaxProblems = 16;
// BN: tile width, one of 16, 64, 256.  cta_pairs != 0 with BN == 256 runs 256 x 256 tiles on CTA pairs.
// order_mode: the order in which the problems' work items are handed out: 0 = heaviest problem first,
// 1 = as listed, 2 = as listed, backwards.
templora_status_t tc_gemm_grouped(const TcProblem *probs, int n, int BN, DeviceStatus *status, cudaStream_t st,
                                  int cta_pairs = 0, int order_mode = 0);
// Decode-time forward of several projections in one launch: clusters of cluster_size (2 or 4) CTAs split
// the k-range of each 128-row tile and sum their partial tiles through distributed shared memory.
// Returns TEMPLORA_ERR_UNSUPPORTED when too few clusters fit (the caller then takes the two-kernel path).
templora_status_t tc_decode_cluster(const TcProblem *probs, int n, int n_tokens, int cluster_size, DeviceStatus *status,
                                    cudaStream_t st);
// Clusters of cluster_size CTAs the one-kernel decode would run on this stream now (0 = not available).
int tc_decode_cluster_count(int cluster_size, int n_tokens, cudaStream_t st);
bool tc_available();
void tc_set_stream_sm_limit(cudaStream_t st, int max_sms);
templora_status_t tc_wait_selftest(DeviceStatus *status, unsigned long long limit_ns, cudaStream_t st);

// ---- workspace need of the decode-time forward alone (api.cu) -------------------
size_t decode_workspace_need(const templora_linear_t *lin, int n);
// The argument checks of templora_decode_fwd that do not involve the workspace.
templora_status_t decode_check_args(const templora_linear_t *lin, int n_tokens, const void *x, const void *y);

}  // namespace templora
