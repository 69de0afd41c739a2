// C-ABI entry points: argument checks, workspace carving and the launch sequences of the
// Temp-Lora chunk update (forward, backward, AdamW, epochs) and of the decode-time forward.
#include "common.cuh"

#include <atomic>
#include <cstring>
#include <utility>
#include <vector>

namespace templora {
namespace {

std::atomic<int> g_kernel_path{0};      // 0 = automatic, 1 = generic kernels only
thread_local int t_path_override = -1;  // set while measuring the workspace needs of both paths

constexpr int kSmRef = 148;  // SM count the split-K heuristic is tuned for (B200)
#ifndef TL_SPLIT_PER_SM
#define TL_SPLIT_PER_SM 3
#endif
#ifndef TL_SPLIT_MIN_KB
#define TL_SPLIT_MIN_KB 8
#endif
#ifndef TL_ORDER_UV
#define TL_ORDER_UV 0
#endif
#ifndef TL_ORDER_GRADS
#define TL_ORDER_GRADS 0
#endif

// Workspace bump allocator.  With base == nullptr it only measures.
struct WsAlloc {
  uint8_t *base;
  size_t off, cap;
  bool overflow = false;
  WsAlloc(void *b, size_t c) : base(reinterpret_cast<uint8_t *>(b)), off(kStatusBytes), cap(c) {}
  template <typename T> T *take(size_t count) {
    size_t bytes = align_up(count * sizeof(T), kWsAlign);
    size_t at = off;
    off += bytes;
    if (!base) return reinterpret_cast<T *>(uintptr_t(kWsAlign));  // dummy non-null
    if (off > cap) { overflow = true; return nullptr; }
    return reinterpret_cast<T *>(base + at);
  }
  DeviceStatus *status() const { return reinterpret_cast<DeviceStatus *>(base); }
};

inline int cdiv(long long a, long long b) { return (int)((a + b - 1) / b); }

// Split-K factor for a skinny problem: `tiles` output tiles, `kb` k-blocks of 64 each, launched
// together with (group-1) similar problems.  Aims at about three work items per SM, never fewer
// than 8 k-blocks per item, at most 16 splits.
int pick_splits(int tiles, int kb, int group) {
  long long total = (long long)tiles * kb * (group < 1 ? 1 : group);
  long long target = (total + kSmRef * TL_SPLIT_PER_SM - 1) / (kSmRef * TL_SPLIT_PER_SM);
  if (target < TL_SPLIT_MIN_KB) target = TL_SPLIT_MIN_KB;
  long long s = (kb + target / 2) / target;
  if (s < 1) s = 1;
  if (s > 16) s = 16;
  if (s > kb) s = kb;
  return (int)s;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

templora_status_t check_linear(const templora_linear_t *lin) {
  if (!lin) return TEMPLORA_ERR_INVALID_ARG;
  if (lin->d_in <= 0 || lin->d_out <= 0 || lin->r <= 0) return TEMPLORA_ERR_INVALID_ARG;
  if (lin->dtype != TEMPLORA_F32 && lin->dtype != TEMPLORA_BF16) return TEMPLORA_ERR_UNSUPPORTED;
  if (lin->r > 256) return TEMPLORA_ERR_UNSUPPORTED;
  if (!(lin->s == lin->s)) return TEMPLORA_ERR_INVALID_ARG;
  if (!(lin->dropout_p >= 0.f && lin->dropout_p < 1.f)) return TEMPLORA_ERR_INVALID_ARG;
  return TEMPLORA_OK;
}
templora_status_t check_linear_ptrs(const templora_linear_t *lin) {
  if (!lin->W0 || !lin->A || !lin->B) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16(lin->W0) || !aligned16(lin->A) || !aligned16(lin->B)) return TEMPLORA_ERR_INVALID_ARG;
  return TEMPLORA_OK;
}
templora_status_t check_ws(const void *ws, size_t ws_bytes) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < kStatusBytes) return TEMPLORA_ERR_WORKSPACE;
  return TEMPLORA_OK;
}

// Does this projection take the tensor-core path?
bool use_tc(const templora_linear_t *lin, bool dry) {
  const int mode = t_path_override >= 0 ? t_path_override : g_kernel_path.load();
  if (mode == 1) return false;
  if (lin->dtype != TEMPLORA_BF16) return false;
  if ((lin->d_in | lin->d_out | lin->r) & 7) return false;
  return dry ? true : tc_available();
}

// Frozen-weight GEMMs on CTA pairs unless kernel path 2 (single-CTA tensor-core tiles) is selected.
int use_pairs() { return g_kernel_path.load() == 2 ? 0 : 1; }

Operand op(const void *p, int dt, long long s0, long long s1) { return Operand{p, dt, s0, s1}; }

// ---------------------------------------------------------------- problem builders (tensor-core path)
TcProblem prob_U(const templora_linear_t *l, int T, const void *x, float *part, int splits) {
  TcProblem p{};
  p.M = T; p.N = l->r; p.K = l->d_in;
  p.A = x; p.lda = l->d_in; p.a_mn = 0;
  p.B = l->A; p.ldb = l->d_in; p.b_mn = 0;
  p.splits = splits; p.out = part; p.out_f32 = 1; p.out_s0 = l->r; p.out_s1 = 1; p.out_split = (long long)T * l->r;
  return p;
}
TcProblem prob_V(const templora_linear_t *l, int T, const void *dY, float *part, int splits) {
  TcProblem p{};
  p.M = T; p.N = l->r; p.K = l->d_out;
  p.A = dY; p.lda = l->d_out; p.a_mn = 0;
  p.B = l->B; p.ldb = l->r; p.b_mn = 1;   // B [d_out, r]: the contraction index d_out is the row index
  p.splits = splits; p.out = part; p.out_f32 = 1; p.out_s0 = l->r; p.out_s1 = 1; p.out_split = (long long)T * l->r;
  return p;
}
TcProblem prob_y(const templora_linear_t *l, int T, const void *x, const void *Us, void *y) {
  TcProblem p{};
  p.M = T; p.N = l->d_out; p.K = l->d_in; p.Kext = l->r;
  p.A = x; p.lda = l->d_in; p.a_mn = 0;
  p.B = l->W0; p.ldb = l->d_in; p.b_mn = 0;
  p.Aext = Us; p.ldaext = l->r; p.Bext = l->B; p.ldbext = l->r;
  p.splits = 1; p.out = y; p.out_f32 = 0; p.out_s0 = l->d_out; p.out_s1 = 1;
  return p;
}
TcProblem prob_dX(const templora_linear_t *l, int T, const void *dY, const void *Vs, void *dX) {
  TcProblem p{};
  p.M = T; p.N = l->d_in; p.K = l->d_out; p.Kext = l->r;
  p.A = dY; p.lda = l->d_out; p.a_mn = 0;
  p.B = l->W0; p.ldb = l->d_in; p.b_mn = 1;    // W0 [d_out, d_in] contracted over its rows
  p.Aext = Vs; p.ldaext = l->r; p.Bext = l->A; p.ldbext = l->d_in;  // A [r, d_in] contracted over its rows
  p.splits = 1; p.out = dX; p.out_f32 = 0; p.out_s0 = l->d_in; p.out_s1 = 1;
  return p;
}
TcProblem prob_dB(const templora_linear_t *l, int T, const void *dY, const void *Us, float *out, int splits) {
  TcProblem p{};
  p.M = l->d_out; p.N = l->r; p.K = T;
  p.A = dY; p.lda = l->d_out; p.a_mn = 1;     // dY^T
  p.B = Us; p.ldb = l->r; p.b_mn = 1;         // Us [T, r] holds s*U
  p.splits = splits; p.out = out; p.out_f32 = 1; p.out_s0 = l->r; p.out_s1 = 1;
  p.out_split = (long long)l->d_out * l->r;
  return p;
}
TcProblem prob_dA(const templora_linear_t *l, int T, const void *x, const void *Vs, float *out, int splits) {
  TcProblem p{};
  p.M = l->d_in; p.N = l->r; p.K = T;         // computes dA^T = x^T (s V), stored transposed
  p.A = x; p.lda = l->d_in; p.a_mn = 1;
  p.B = Vs; p.ldb = l->r; p.b_mn = 1;
  p.splits = splits; p.out = out; p.out_f32 = 1; p.out_s0 = 1; p.out_s1 = l->d_in;
  p.out_split = (long long)l->d_in * l->r;
  return p;
}

int splits_skinny(int T, int r, int K, int group) { return pick_splits(cdiv(T, 128) * cdiv(r, 64), cdiv(K, 64), group); }
int splits_grad(int d, int r, int T, int group) { return pick_splits(cdiv(d, 128) * cdiv(r, 64), cdiv(T, 64), group); }

// ---------------------------------------------------------------- dropout scratch
struct DropBufs {
  void *xd = nullptr;        // x * keep / (1 - p), storage type of x
  uint8_t *mask = nullptr;   // keep bits
  long long pitch = 0;
};
DropBufs take_drop(const templora_linear_t *l, int T, WsAlloc &ws) {
  DropBufs d;
  if (l->dropout_p > 0.f) {
    const size_t esize = l->dtype == TEMPLORA_BF16 ? 2 : 4;
    d.xd = ws.take<uint8_t>((size_t)T * l->d_in * esize);
    d.pitch = dropout_mask_pitch(l->d_in);
    d.mask = ws.take<uint8_t>((size_t)T * d.pitch);
  }
  return d;
}
DropoutJob drop_job(const templora_linear_t *l, int T, const void *x, const DropBufs &d, uint64_t step_offset) {
  return DropoutJob{x, d.xd, d.mask, T, l->d_in, d.pitch, l->dtype, l->dropout_p, l->dropout_seed,
                    l->dropout_offset + step_offset};
}
// dX += keep * (s / (1 - p)) * (V A): one pass over dX on 128 x 256 tiles with a single k-block
TcProblem prob_dX_dropout_term(const templora_linear_t *l, int T, const void *Vs, void *dX, const DropBufs &d) {
  TcProblem p{};
  p.M = T; p.N = l->d_in; p.K = l->r;
  p.A = Vs; p.lda = l->r; p.a_mn = 0;
  p.B = l->A; p.ldb = l->d_in; p.b_mn = 1;
  p.splits = 1; p.out = dX; p.out_f32 = 0; p.out_s0 = l->d_in; p.out_s1 = 1;
  p.epi_mask = d.mask; p.epi_mask_pitch = d.pitch; p.epi_scale = (float)(1.0 / (1.0 - (double)l->dropout_p));
  return p;
}

// ---------------------------------------------------------------- forward
templora_status_t fwd_impl(const templora_linear_t *l, int T, const void *x, void *y, float *U_save, WsAlloc &ws,
                           bool dry, cudaStream_t st) {
  const long long Tr = (long long)T * l->r;
  if (use_tc(l, dry)) {
    const int su = splits_skinny(T, l->r, l->d_in, 1);
    float *Upart = ws.take<float>((size_t)su * Tr);
    __nv_bfloat16 *Us = ws.take<__nv_bfloat16>((size_t)Tr);
    const DropBufs drop = take_drop(l, T, ws);
    if (dry) return TEMPLORA_OK;
    if (ws.overflow) return TEMPLORA_ERR_WORKSPACE;
    if (drop.xd) {
      DropoutJob dj = drop_job(l, T, x, drop, 0);
      TL_TRY(dropout_apply_batch(&dj, 1, st));
    }
    TcProblem pu = prob_U(l, T, drop.xd ? drop.xd : x, Upart, su);
    TL_TRY(tc_gemm_grouped(&pu, 1, 64, ws.status(), st));
    ReduceJob rj{Upart, su, Tr, Tr, l->s, 1.f, U_save, 0, Us};
    TL_TRY(reduce_partials_batch(&rj, 1, st));
    TcProblem py = prob_y(l, T, x, Us, y);
    return tc_gemm_grouped(&py, 1, 256, ws.status(), st, use_pairs());
  }
  float *U = U_save ? U_save : ws.take<float>((size_t)Tr);
  const DropBufs drop = take_drop(l, T, ws);
  if (dry) return TEMPLORA_OK;
  if (ws.overflow) return TEMPLORA_ERR_WORKSPACE;
  const int dt = l->dtype;
  if (drop.xd) {
    DropoutJob dj = drop_job(l, T, x, drop, 0);
    TL_TRY(dropout_apply_batch(&dj, 1, st));
  }
  SimtGemm g{};
  g.M = T; g.N = l->r; g.K1 = l->d_in; g.K2 = 0;
  g.A1 = op(drop.xd ? drop.xd : x, dt, l->d_in, 1); g.B1 = op(l->A, dt, 1, l->d_in);
  g.alpha1 = 1.f; g.alpha2 = 0.f; g.D = U; g.d_dt = TEMPLORA_F32; g.ds0 = l->r; g.ds1 = 1;
  TL_TRY(simt_gemm(g, st));
  SimtGemm h{};
  h.M = T; h.N = l->d_out; h.K1 = l->d_in; h.K2 = l->r;
  h.A1 = op(x, dt, l->d_in, 1); h.B1 = op(l->W0, dt, 1, l->d_in);
  h.A2 = op(U, TEMPLORA_F32, l->r, 1); h.B2 = op(l->B, dt, 1, l->r);
  h.alpha1 = 1.f; h.alpha2 = l->s; h.D = y; h.d_dt = dt; h.ds0 = l->d_out; h.ds1 = 1;
  return simt_gemm(h, st);
}

// ---------------------------------------------------------------- backward
templora_status_t bwd_impl(const templora_linear_t *l, int T, const void *x, const void *dY, const float *U_saved,
                           void *dX, float *dA, float *dB, int accumulate, WsAlloc &ws, bool dry, cudaStream_t st,
                           int dx_accumulate = 0) {
  const long long Tr = (long long)T * l->r;
  if (dx_accumulate && use_tc(l, dry)) return TEMPLORA_ERR_UNSUPPORTED;   // summed dX: grouped path or generic kernels
  if (use_tc(l, dry)) {
    const int su = U_saved ? 1 : splits_skinny(T, l->r, l->d_in, 2);
    const int sv = splits_skinny(T, l->r, l->d_out, 2);
    const int sb = splits_grad(l->d_out, l->r, T, 2), sa = splits_grad(l->d_in, l->r, T, 2);
    float *Upart = U_saved ? nullptr : ws.take<float>((size_t)su * Tr);
    float *Vpart = ws.take<float>((size_t)sv * Tr);
    __nv_bfloat16 *Us = ws.take<__nv_bfloat16>((size_t)Tr);
    __nv_bfloat16 *Vs = ws.take<__nv_bfloat16>((size_t)Tr);
    const bool direct_b = (sb == 1 && !accumulate), direct_a = (sa == 1 && !accumulate);
    float *dBpart = direct_b ? dB : ws.take<float>((size_t)sb * l->d_out * l->r);
    float *dApart = direct_a ? dA : ws.take<float>((size_t)sa * l->d_in * l->r);
    const DropBufs drop = take_drop(l, T, ws);
    if (dry) return TEMPLORA_OK;
    if (ws.overflow) return TEMPLORA_ERR_WORKSPACE;
    if (drop.xd) {   // the same mask as the forward's: same seed, same offset, same shape
      DropoutJob dj = drop_job(l, T, x, drop, 0);
      TL_TRY(dropout_apply_batch(&dj, 1, st));
    }
    const void *xb = drop.xd ? drop.xd : x;   // what the low-rank branch read

    TcProblem skinny[2];
    int ns = 0;
    skinny[ns++] = prob_V(l, T, dY, Vpart, sv);
    if (!U_saved) skinny[ns++] = prob_U(l, T, xb, Upart, su);
    TL_TRY(tc_gemm_grouped(skinny, ns, 64, ws.status(), st));
    ReduceJob jobs[2] = {
        ReduceJob{Vpart, sv, Tr, Tr, l->s, 1.f, nullptr, 0, Vs},
        ReduceJob{U_saved ? U_saved : Upart, su, Tr, Tr, l->s, 1.f, nullptr, 0, Us},
    };
    TL_TRY(reduce_partials_batch(jobs, 2, st));
    if (dX) {
      TcProblem px = prob_dX(l, T, dY, Vs, dX);
      if (drop.xd) px.Kext = 0;   // the rank-r term is masked per element: added by a second pass
      TL_TRY(tc_gemm_grouped(&px, 1, 256, ws.status(), st, use_pairs()));
      if (drop.xd) {
        TcProblem pt = prob_dX_dropout_term(l, T, Vs, dX, drop);
        TL_TRY(tc_gemm_grouped(&pt, 1, 256, ws.status(), st, 0));
      }
    }
    TcProblem grads[2] = {prob_dB(l, T, dY, Us, dBpart, sb), prob_dA(l, T, xb, Vs, dApart, sa)};
    TL_TRY(tc_gemm_grouped(grads, 2, 64, ws.status(), st));
    ReduceJob rj[2];
    int nr = 0;
    const long long nb = (long long)l->d_out * l->r, na = (long long)l->d_in * l->r;
    if (!direct_b) rj[nr++] = ReduceJob{dBpart, sb, nb, nb, 1.f, 1.f, dB, accumulate, nullptr};
    if (!direct_a) rj[nr++] = ReduceJob{dApart, sa, na, na, 1.f, 1.f, dA, accumulate, nullptr};
    if (nr) TL_TRY(reduce_partials_batch(rj, nr, st));
    return TEMPLORA_OK;
  }
  float *Ubuf = U_saved ? nullptr : ws.take<float>((size_t)Tr);
  float *V = ws.take<float>((size_t)Tr);
  const DropBufs drop = take_drop(l, T, ws);
  if (dry) return TEMPLORA_OK;
  if (ws.overflow) return TEMPLORA_ERR_WORKSPACE;
  const int dt = l->dtype;
  if (drop.xd) {
    DropoutJob dj = drop_job(l, T, x, drop, 0);
    TL_TRY(dropout_apply_batch(&dj, 1, st));
  }
  const void *xb = drop.xd ? drop.xd : x;
  const float *U = U_saved;
  if (!U) {
    SimtGemm g{};
    g.M = T; g.N = l->r; g.K1 = l->d_in;
    g.A1 = op(xb, dt, l->d_in, 1); g.B1 = op(l->A, dt, 1, l->d_in);
    g.alpha1 = 1.f; g.D = Ubuf; g.d_dt = TEMPLORA_F32; g.ds0 = l->r; g.ds1 = 1;
    TL_TRY(simt_gemm(g, st));
    U = Ubuf;
  }
  {  // V = dY B
    SimtGemm g{};
    g.M = T; g.N = l->r; g.K1 = l->d_out;
    g.A1 = op(dY, dt, l->d_out, 1); g.B1 = op(l->B, dt, l->r, 1);
    g.alpha1 = 1.f; g.D = V; g.d_dt = TEMPLORA_F32; g.ds0 = l->r; g.ds1 = 1;
    TL_TRY(simt_gemm(g, st));
  }
  if (dX && !drop.xd) {  // dX = dY W0 + s V A
    SimtGemm g{};
    g.M = T; g.N = l->d_in; g.K1 = l->d_out; g.K2 = l->r;
    g.A1 = op(dY, dt, l->d_out, 1); g.B1 = op(l->W0, dt, l->d_in, 1);
    g.A2 = op(V, TEMPLORA_F32, l->r, 1); g.B2 = op(l->A, dt, l->d_in, 1);
    g.alpha1 = 1.f; g.alpha2 = l->s; g.D = dX; g.d_dt = dt; g.ds0 = l->d_in; g.ds1 = 1; g.accumulate = dx_accumulate;
    TL_TRY(simt_gemm(g, st));
  }
  if (dX && drop.xd) {  // dX = dY W0, then dX += keep * s / (1 - p) * (V A)
    SimtGemm g{};
    g.M = T; g.N = l->d_in; g.K1 = l->d_out;
    g.A1 = op(dY, dt, l->d_out, 1); g.B1 = op(l->W0, dt, l->d_in, 1);
    g.alpha1 = 1.f; g.D = dX; g.d_dt = dt; g.ds0 = l->d_in; g.ds1 = 1; g.accumulate = dx_accumulate;
    TL_TRY(simt_gemm(g, st));
    SimtGemm h{};
    h.M = T; h.N = l->d_in; h.K1 = l->r;
    h.A1 = op(V, TEMPLORA_F32, l->r, 1); h.B1 = op(l->A, dt, l->d_in, 1);
    h.alpha1 = (float)((double)l->s / (1.0 - (double)l->dropout_p));
    h.D = dX; h.d_dt = dt; h.ds0 = l->d_in; h.ds1 = 1; h.accumulate = 1; h.mask = drop.mask; h.mask_pitch = drop.pitch;
    TL_TRY(simt_gemm(h, st));
  }
  {  // dB = s dY^T U
    SimtGemm g{};
    g.M = l->d_out; g.N = l->r; g.K1 = T;
    g.A1 = op(dY, dt, 1, l->d_out); g.B1 = op(U, TEMPLORA_F32, l->r, 1);
    g.alpha1 = l->s; g.D = dB; g.d_dt = TEMPLORA_F32; g.ds0 = l->r; g.ds1 = 1; g.accumulate = accumulate;
    TL_TRY(simt_gemm(g, st));
  }
  {  // dA = s V^T x
    SimtGemm g{};
    g.M = l->r; g.N = l->d_in; g.K1 = T;
    g.A1 = op(V, TEMPLORA_F32, 1, l->r); g.B1 = op(xb, dt, l->d_in, 1);
    g.alpha1 = l->s; g.D = dA; g.d_dt = TEMPLORA_F32; g.ds0 = l->d_in; g.ds1 = 1; g.accumulate = accumulate;
    TL_TRY(simt_gemm(g, st));
  }
  return TEMPLORA_OK;
}

// ---------------------------------------------------------------- decode
// Finish of the decode-time forward, for up to kDecGroup projections in one launch:
//   y[i,o] = sum_k P[k][i][o] + s * sum_j (sum_k Pu[k][i][j]) * B[o][j]
// P, Pu are the split-K partial slabs of W0 x^T and A x^T written by the tensor-core kernel; the
// rank-r term is added in registers.
constexpr int kDecGroup = 8;
struct FinishEntry {
  const float *P, *Pu;
  const __nv_bfloat16 *B;
  __nv_bfloat16 *y;
  int sp, spu, d_out, r, block_start;
  float s;
};
struct FinishBatch {
  FinishEntry e[kDecGroup];
  int n_entries, n_tokens;
};

// Block = kFinO output features x TY token lanes.  The block first stages its kFinO rows of B in
// shared memory with coalesced loads (row pitch padded by 16 bytes: conflict-free row-per-thread
// reads) and the scaled u = s * (A x^T) of all tokens; then thread (o, ty) finishes tokens ty, ty+TY, ...
constexpr int kFinO = 64;
constexpr int kFinTy = 4;   // 256 threads per block: the whole grid (d_out / 64 blocks) is resident at once

// TOK = tokens per thread: 1 when n <= kFinTy (every token has its own lane), else 4.
template <int TOK>
__global__ void __launch_bounds__(kFinO * kFinTy, 6) decode_finish_kernel(const __grid_constant__ FinishBatch fb) {
  extern __shared__ __align__(16) uint8_t fin_smem[];
  pdl_prologue();
  int j = 0;
  while (j + 1 < fb.n_entries && (int)blockIdx.x >= fb.e[j + 1].block_start) ++j;
  const FinishEntry &f = fb.e[j];
  const int n = fb.n_tokens, r = f.r, d_out = f.d_out;
  const int pitch = r + 8;                                        // bf16 elements per staged row of B
  __nv_bfloat16 *b_sm = reinterpret_cast<__nv_bfloat16 *>(fin_smem);
  float *u_sm = reinterpret_cast<float *>(fin_smem + (size_t)kFinO * pitch * 2);   // [n][r]
  const int tid = threadIdx.y * kFinO + threadIdx.x, nthreads = kFinO * blockDim.y;
  const int o0 = (blockIdx.x - f.block_start) * kFinO;

  // stage B[o0 .. o0+kFinO) x r (16-byte chunks, coalesced along r)
  const int chunks_per_row = r >> 3;
  for (int c = tid; c < kFinO * chunks_per_row; c += nthreads) {
    const int row = c / chunks_per_row, ch = c - row * chunks_per_row;
    uint4 w = make_uint4(0, 0, 0, 0);
    if (o0 + row < d_out) w = *reinterpret_cast<const uint4 *>(f.B + (long long)(o0 + row) * r + ch * 8);
    *reinterpret_cast<uint4 *>(b_sm + row * pitch + ch * 8) = w;
  }
  for (int e0 = tid; e0 < n * r; e0 += 4 * nthreads) {   // four elements per thread per pass, loads batched
    float a[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k = 0; k < f.spu; ++k) {
      const float *src = f.Pu + (long long)k * n * r;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int e = e0 + q * nthreads;
        if (e < n * r) a[q] += __ldg(src + e);
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int e = e0 + q * nthreads;
      if (e < n * r) u_sm[e] = f.s * a[q];
    }
  }
  __syncthreads();
  const int o = o0 + threadIdx.x;
  if (o >= d_out) return;
  const __nv_bfloat16 *brow = b_sm + threadIdx.x * pitch;
  // tokens threadIdx.y, +kFinTy, ... (at most four): all their slab loads are issued before any is used,
  // so the slabs (usually evicted to DRAM by the W0 stream) cost one memory latency per slab, not per token
  float acc[TOK];
#pragma unroll
  for (int q = 0; q < TOK; ++q) acc[q] = 0.f;
  for (int k = 0; k < f.sp; ++k) {
    const float *src = f.P + (long long)k * n * d_out + o;
    float t[TOK];
#pragma unroll
    for (int q = 0; q < TOK; ++q) {
      const int i = threadIdx.y + q * kFinTy;
      t[q] = (i < n) ? __ldg(src + (long long)i * d_out) : 0.f;
    }
#pragma unroll
    for (int q = 0; q < TOK; ++q) acc[q] += t[q];
  }
  for (int j0 = 0; j0 < r; j0 += 8) {
    const uint4 w = *reinterpret_cast<const uint4 *>(brow + j0);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&w);
    const float2 b0 = __bfloat1622float2(h[0]), b1 = __bfloat1622float2(h[1]);
    const float2 b2 = __bfloat1622float2(h[2]), b3 = __bfloat1622float2(h[3]);
#pragma unroll
    for (int q = 0; q < TOK; ++q) {
      const int i = threadIdx.y + q * kFinTy;
      if (i < n) {
        const float *urow = u_sm + i * r + j0;
        const float4 u0 = *reinterpret_cast<const float4 *>(urow);       // same address across the warp
        const float4 u1 = *reinterpret_cast<const float4 *>(urow + 4);
        float a = acc[q];
        a = fmaf(u0.x, b0.x, a); a = fmaf(u0.y, b0.y, a); a = fmaf(u0.z, b1.x, a); a = fmaf(u0.w, b1.y, a);
        a = fmaf(u1.x, b2.x, a); a = fmaf(u1.y, b2.y, a); a = fmaf(u1.z, b3.x, a); a = fmaf(u1.w, b3.y, a);
        acc[q] = a;
      }
    }
  }
#pragma unroll
  for (int q = 0; q < TOK; ++q) {
    const int i = threadIdx.y + q * kFinTy;
    if (i < n) f.y[(long long)i * d_out + o] = __float2bfloat16_rn(acc[q]);
  }
}

// Split-K factor of the decode stream of one projection launched together with others whose
// k-blocks add up to total_kb.  Few tokens: about 12 work items per SM (short tail, the partial
// slabs are tiny); many tokens: about 6 (the slabs grow with the token count).  Never fewer than
// 8 k-blocks per item.
int decode_splits(int kb, long long total_kb, int n) {
  const int per_sm = n <= 4 ? 12 : 6;
  long long target = (total_kb + kSmRef * per_sm - 1) / (kSmRef * per_sm);
  if (target < 8) target = 8;
  long long s = (kb + target / 2) / target;
  if (s < 1) s = 1;
  if (s > 16) s = 16;
  if (s > kb) s = kb;
  return (int)s;
}
// Rows of partial sums to reserve per output feature so that any token count 1..16 fits.
int decode_partial_rows(int kb, long long total_kb) {
  const int a = decode_splits(kb, total_kb, 4) * 4, b = decode_splits(kb, total_kb, 16) * 16;
  return a > b ? a : b;
}

// Cluster size (CTAs that split the k-range of one 128-row tile) for the one-kernel decode of a group:
// the candidate whose list schedule (items in launch order, each to the cluster that frees up first)
// ends soonest.  An item costs a cluster of S its k-blocks per CTA plus a fixed hand-over cost (measured:
// about five k-blocks' worth), and the launched CTAs share the memory bandwidth.  0 = none applies.
int decode_cluster_size_search(const templora_linear_t *proj, int np, int n, cudaStream_t st);
// The search costs tens of microseconds of host time and a decode call only a few: the answer is
// remembered per thread by the shapes it was found for (and by the cluster counts, which a per-stream
// SM cap changes).
int decode_cluster_size(const templora_linear_t *proj, int np, int n, cudaStream_t st) {
  struct Key {
    int np, n, c2, c4, dims[3 * kDecGroup];
    bool operator==(const Key &o) const { return memcmp(this, &o, sizeof(Key)) == 0; }
  };
  static thread_local std::vector<std::pair<Key, int>> cache;
  Key k;
  memset(&k, 0, sizeof(k));
  k.np = np; k.n = n; k.c2 = tc_decode_cluster_count(2, n, st); k.c4 = tc_decode_cluster_count(4, n, st);
  for (int i = 0; i < np; ++i) { k.dims[3 * i] = proj[i].d_in; k.dims[3 * i + 1] = proj[i].d_out; k.dims[3 * i + 2] = proj[i].r; }
  for (const auto &e : cache)
    if (e.first == k) return e.second;
  const int S = decode_cluster_size_search(proj, np, n, st);
  if (cache.size() >= 256) cache.clear();
  cache.emplace_back(k, S);
  return S;
}
int decode_cluster_size_search(const templora_linear_t *proj, int np, int n, cudaStream_t st) {
  const int cand[2] = {2, 4};
  int best = 0;
  double best_t = 0.0;
  for (int c = 0; c < 2; ++c) {
    const int S = cand[c], clusters = tc_decode_cluster_count(S, n, st);
    bool fits = clusters >= np;
    for (int i = 0; i < np; ++i) fits = fits && cdiv(proj[i].d_in, 64) >= S;
    if (!fits) continue;
    std::vector<double> load(clusters, 0.0);
    auto give = [&](double w) {
      int k = 0;
      for (int j = 1; j < clusters; ++j) if (load[j] < load[k]) k = j;
      load[k] += w;
    };
    const double hand_over = 5.0;
    for (int i = 0; i < np; ++i) give((double)cdiv(proj[i].d_in, 64) / S + hand_over);
    int order[kDecGroup];   // the launch deals the projections with the longest k-range first
    for (int i = 0; i < np; ++i) order[i] = i;
    for (int i = 1; i < np; ++i)
      for (int j = i; j > 0 && proj[order[j]].d_in > proj[order[j - 1]].d_in; --j) std::swap(order[j], order[j - 1]);
    for (int k = 0; k < np; ++k) {
      const templora_linear_t &l = proj[order[k]];
      const double w = (double)(cdiv(l.d_in, 64) + cdiv(l.r, 64)) / S + hand_over;
      for (int t = 0; t < cdiv(l.d_out, 128); ++t) give(w);
    }
    double span = 0.0;
    for (double l : load) span = l > span ? l : span;
    const double t = span * S * clusters;
    if (best == 0 || t < best_t) { best = S; best_t = t; }
  }
  return best;
}

// One-kernel decode of a group: per projection a u problem (A x^T, stored as bf16(s u)) and a y problem
// (W0 x^T with the rank-r term as extension k-blocks B (s u)^T).  su: np buffers of 16 * r bf16.
templora_status_t decode_group_cluster(const templora_linear_t *proj, int np, int n, const void *const *x,
                                       void *const *y, __nv_bfloat16 *const *su, int S, DeviceStatus *status,
                                       cudaStream_t st) {
  TcProblem p[2 * kDecGroup] = {};
  // y problems heaviest first; u problems lead the launch
  int order[kDecGroup];
  for (int i = 0; i < np; ++i) order[i] = i;
  for (int i = 1; i < np; ++i)
    for (int j = i; j > 0 && proj[order[j]].d_in > proj[order[j - 1]].d_in; --j) std::swap(order[j], order[j - 1]);
  for (int k = 0; k < np; ++k) {
    const int i = order[k];
    const templora_linear_t *l = proj + i;
    TcProblem &u = p[k], &a = p[np + k];
    u.M = l->r; u.N = n; u.K = l->d_in;
    u.A = l->A; u.lda = l->d_in; u.B = x[i]; u.ldb = l->d_in;
    u.splits = 1; u.out = su[i]; u.out_s0 = 1; u.out_s1 = l->r; u.epi_scale = l->s; u.role = 1; u.flag = k;
    a.M = l->d_out; a.N = n; a.K = l->d_in; a.Kext = l->r;
    a.A = l->W0; a.lda = l->d_in; a.B = x[i]; a.ldb = l->d_in;
    a.Aext = l->B; a.ldaext = l->r; a.Bext = su[i]; a.ldbext = l->r;
    a.splits = 1; a.out = y[i]; a.out_s0 = 1; a.out_s1 = l->d_out; a.epi_scale = 1.f; a.role = 0; a.flag = k;
  }
  return tc_decode_cluster(p, 2 * np, n, S, status, st);
}

// Decode-time forward of up to kDecGroup projections (all on the tensor-core path): one grouped
// launch streams every W0 and A once, one launch finishes.
templora_status_t decode_group_tc(const templora_linear_t *proj, int np, int n, const void *const *x, void *const *y,
                                  WsAlloc &ws, bool dry, cudaStream_t st) {
  long long total_kb = 0;
  for (int i = 0; i < np; ++i)
    total_kb += (long long)(cdiv(proj[i].d_out, 128) + cdiv(proj[i].r, 128)) * cdiv(proj[i].d_in, 64);
  TcProblem p[2 * kDecGroup] = {};
  FinishBatch fb;
  fb.n_entries = np; fb.n_tokens = n;
  int blocks = 0, max_r = 0;
  __nv_bfloat16 *su[kDecGroup];
  for (int i = 0; i < np; ++i) su[i] = ws.take<__nv_bfloat16>((size_t)16 * proj[i].r);
  if (!dry && use_pairs()) {   // kernel path 2 keeps the two-kernel form below
    if (ws.overflow) return TEMPLORA_ERR_WORKSPACE;
    const int S = decode_cluster_size(proj, np, n, st);
    if (S > 0) {
      const templora_status_t rc = decode_group_cluster(proj, np, n, x, y, su, S, ws.status(), st);
      if (rc != TEMPLORA_ERR_UNSUPPORTED) return rc;
    }
  }
  for (int i = 0; i < np; ++i) {
    const templora_linear_t *l = proj + i;
    const int kb = cdiv(l->d_in, 64);
    const int sp = decode_splits(kb, total_kb, n), spu = sp;
    const int rows = decode_partial_rows(kb, total_kb);
    float *P = ws.take<float>((size_t)rows * l->d_out);
    float *Pu = ws.take<float>((size_t)rows * l->r);
    if (dry) continue;
    if (ws.overflow) return TEMPLORA_ERR_WORKSPACE;
    TcProblem &a = p[2 * i], &u = p[2 * i + 1];
    a.M = l->d_out; a.N = n; a.K = l->d_in;
    a.A = l->W0; a.lda = l->d_in; a.B = x[i]; a.ldb = l->d_in;
    a.splits = sp; a.out = P; a.out_f32 = 1; a.out_s0 = 1; a.out_s1 = l->d_out; a.out_split = (long long)n * l->d_out;
    u.M = l->r; u.N = n; u.K = l->d_in;
    u.A = l->A; u.lda = l->d_in; u.B = x[i]; u.ldb = l->d_in;
    u.splits = spu; u.out = Pu; u.out_f32 = 1; u.out_s0 = 1; u.out_s1 = l->r; u.out_split = (long long)n * l->r;
    fb.e[i] = FinishEntry{P, Pu, reinterpret_cast<const __nv_bfloat16 *>(l->B), reinterpret_cast<__nv_bfloat16 *>(y[i]),
                          sp, spu, l->d_out, l->r, blocks, l->s};
    blocks += cdiv(l->d_out, kFinO);
    if (l->r > max_r) max_r = l->r;
  }
  if (dry) return TEMPLORA_OK;
  TL_TRY(tc_gemm_grouped(p, 2 * np, 16, ws.status(), st));
  {
    LaunchScope scope(kKindDecodeFinish, st);
    const size_t smem = (size_t)kFinO * (max_r + 8) * 2 + (size_t)n * max_r * sizeof(float);
    static bool attr_done_dev[64] = {};   // function attributes are per device
    int dev_id = 0;
    TL_CUDA_CHECK(cudaGetDevice(&dev_id));
    bool &attr_done = attr_done_dev[dev_id & 63];
    if (!attr_done) {
      TL_CUDA_CHECK(cudaFuncSetAttribute(decode_finish_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
      TL_CUDA_CHECK(cudaFuncSetAttribute(decode_finish_kernel<1>, cudaFuncAttributePreferredSharedMemoryCarveout, 50));
      TL_CUDA_CHECK(cudaFuncSetAttribute(decode_finish_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
      TL_CUDA_CHECK(cudaFuncSetAttribute(decode_finish_kernel<4>, cudaFuncAttributePreferredSharedMemoryCarveout, 50));
      attr_done = true;
    }
    if (n <= kFinTy)
      TL_CUDA_CHECK(launch_pdl(decode_finish_kernel<1>, dim3(blocks), dim3(kFinO, kFinTy), smem, st, fb));
    else
      TL_CUDA_CHECK(launch_pdl(decode_finish_kernel<4>, dim3(blocks), dim3(kFinO, kFinTy), smem, st, fb));
  }
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

templora_status_t decode_impl(const templora_linear_t *l, int n, const void *x, void *y, WsAlloc &ws, bool dry,
                              cudaStream_t st) {
  if (use_tc(l, dry)) return decode_group_tc(l, 1, n, &x, &y, ws, dry, st);
  return fwd_impl(l, n, x, y, nullptr, ws, dry, st);
}

// Several independent projections in one call.  Groups of kDecGroup run one after another on the
// stream and reuse the same workspace region.
templora_status_t decode_block_impl(const templora_linear_t *proj, int n_proj, int n, const void *const *x,
                                    void *const *y, void *ws_ptr, size_t ws_bytes, bool dry, size_t *need,
                                    cudaStream_t st) {
  size_t max_need = kStatusBytes;
  int i = 0;
  while (i < n_proj) {
    WsAlloc a(dry ? nullptr : ws_ptr, ws_bytes);
    if (use_tc(proj + i, dry)) {
      int np = 1;
      while (i + np < n_proj && np < kDecGroup && use_tc(proj + i + np, dry)) ++np;
      TL_TRY(decode_group_tc(proj + i, np, n, dry ? nullptr : x + i, dry ? nullptr : y + i, a, dry, st));
      i += np;
    } else {
      TL_TRY(fwd_impl(proj + i, n, dry ? nullptr : x[i], dry ? nullptr : y[i], nullptr, a, dry, st));
      i += 1;
    }
    if (a.off > max_need) max_need = a.off;
  }
  if (need) *need = max_need;
  return TEMPLORA_OK;
}

// ---------------------------------------------------------------- update_block (tensor-core, grouped)
constexpr int kGroup = 8;  // projections per grouped launch (two problems each)

struct GroupBufs {
  float *Upart[kGroup], *Vpart[kGroup], *dBpart[kGroup], *dApart[kGroup];
  __nv_bfloat16 *Us[kGroup], *Vs[kGroup];
  int su[kGroup], sv[kGroup], sb[kGroup], sa[kGroup];
  DropBufs drop[kGroup];
};

void carve_group(const templora_linear_t *proj, int n, int T, WsAlloc &ws, GroupBufs &b) {
  for (int i = 0; i < n; ++i) {
    const templora_linear_t *l = proj + i;
    const long long Tr = (long long)T * l->r;
    b.su[i] = splits_skinny(T, l->r, l->d_in, 2 * n);
    b.sv[i] = splits_skinny(T, l->r, l->d_out, 2 * n);
    b.sb[i] = splits_grad(l->d_out, l->r, T, 2 * n);
    b.sa[i] = splits_grad(l->d_in, l->r, T, 2 * n);
    b.Upart[i] = ws.take<float>((size_t)b.su[i] * Tr);
    b.Vpart[i] = ws.take<float>((size_t)b.sv[i] * Tr);
    b.Us[i] = ws.take<__nv_bfloat16>((size_t)Tr);
    b.Vs[i] = ws.take<__nv_bfloat16>((size_t)Tr);
    b.dBpart[i] = b.sb[i] > 1 ? ws.take<float>((size_t)b.sb[i] * l->d_out * l->r) : nullptr;
    b.dApart[i] = b.sa[i] > 1 ? ws.take<float>((size_t)b.sa[i] * l->d_in * l->r) : nullptr;
    b.drop[i] = take_drop(l, T, ws);
  }
}

templora_status_t update_group_tc(const templora_linear_t *proj, const templora_param_t *As, const templora_param_t *Bs,
                                  int n, int T, const void *const *x, const void *const *dY, void *const *y,
                                  void *const *dX, const GroupBufs &b, DeviceStatus *status, uint64_t steps_taken,
                                  cudaStream_t st) {
  TcProblem probs[2 * kGroup];
  ReduceJob jobs[2 * kGroup];
  DropoutJob drops[kGroup];
  const void *xb[kGroup];   // what the low-rank branch reads: x, or x with this step's dropout applied
  int np = 0, nj = 0, nd = 0;
  for (int i = 0; i < n; ++i) {
    xb[i] = x[i];
    if (b.drop[i].xd) {
      drops[nd++] = drop_job(proj + i, T, x[i], b.drop[i], steps_taken);
      xb[i] = b.drop[i].xd;
    }
  }
  if (nd) TL_TRY(dropout_apply_batch(drops, nd, st));
  for (int i = 0; i < n; ++i) {
    const long long Tr = (long long)T * proj[i].r;
    probs[np++] = prob_U(proj + i, T, xb[i], b.Upart[i], b.su[i]);
    probs[np++] = prob_V(proj + i, T, dY[i], b.Vpart[i], b.sv[i]);
    jobs[nj++] = ReduceJob{b.Upart[i], b.su[i], Tr, Tr, proj[i].s, 1.f, nullptr, 0, b.Us[i]};
    jobs[nj++] = ReduceJob{b.Vpart[i], b.sv[i], Tr, Tr, proj[i].s, 1.f, nullptr, 0, b.Vs[i]};
  }
  TL_TRY(tc_gemm_grouped(probs, np, 64, status, st, 0, TL_ORDER_UV));
  TL_TRY(reduce_partials_batch(jobs, nj, st));
  // dB and dA go before the frozen-weight GEMMs: they re-read x and dY, which the U, V launch has just
  // pulled through L2 (the big GEMMs stream 1.1 GB and would flush them)
  auto launch_grads = [&]() -> templora_status_t {
    np = 0; nj = 0;
    for (int i = 0; i < n; ++i) {
      const templora_linear_t *l = proj + i;
      float *gB = const_cast<float *>(Bs[i].grad), *gA = const_cast<float *>(As[i].grad);
      probs[np++] = prob_dB(l, T, dY[i], b.Us[i], b.sb[i] > 1 ? b.dBpart[i] : gB, b.sb[i]);
      probs[np++] = prob_dA(l, T, xb[i], b.Vs[i], b.sa[i] > 1 ? b.dApart[i] : gA, b.sa[i]);
      const long long nb = (long long)l->d_out * l->r, na = (long long)l->d_in * l->r;
      if (b.sb[i] > 1) jobs[nj++] = ReduceJob{b.dBpart[i], b.sb[i], nb, nb, 1.f, 1.f, gB, 0, nullptr};
      if (b.sa[i] > 1) jobs[nj++] = ReduceJob{b.dApart[i], b.sa[i], na, na, 1.f, 1.f, gA, 0, nullptr};
    }
    TL_TRY(tc_gemm_grouped(probs, np, 64, status, st, 0, TL_ORDER_GRADS));
    if (nj) TL_TRY(reduce_partials_batch(jobs, nj, st));
    return TEMPLORA_OK;
  };
  auto launch_main = [&]() -> templora_status_t {
    np = 0;
    // Projections given the same dX buffer (they share their input) get ONE problem: the products of the
    // later ones are appended to the first one's k-loop, so the sum forms in the accumulator.
    int owner[kGroup], rank_in_set[kGroup], prob_of[kGroup], max_rank = 0;
    for (int i = 0; i < n; ++i) {
      owner[i] = i; rank_in_set[i] = 0; prob_of[i] = -1;
      if (!(dX && dX[i])) continue;
      for (int k = 0; k < i && proj[i].input_group != 0; ++k)
        if (dX[k] && proj[k].input_group == proj[i].input_group) { owner[i] = owner[k]; ++rank_in_set[i]; }
      if (rank_in_set[i] > max_rank) max_rank = rank_in_set[i];
    }
    for (int i = 0; i < n; ++i) {
      probs[np++] = prob_y(proj + i, T, x[i], b.Us[i], y[i]);
      if (!(dX && dX[i])) continue;
      if (owner[i] == i) {
        prob_of[i] = np;
        probs[np] = prob_dX(proj + i, T, dY[i], b.Vs[i], dX[i]);
        if (b.drop[i].xd) probs[np].Kext = 0;   // masked rank-r term: second pass below
        ++np;
      } else {
        TcProblem &o = probs[prob_of[owner[i]]];
        if (proj[i].d_in != proj[owner[i]].d_in || o.n_extra + 2 > 4) return TEMPLORA_ERR_INVALID_ARG;
        int e = o.n_extra;
        o.Ax[e] = dY[i]; o.ldax[e] = proj[i].d_out; o.Bx[e] = proj[i].W0; o.ldbx[e] = proj[i].d_in; o.Kx[e] = proj[i].d_out;
        ++e;
        if (!b.drop[i].xd) {
          o.Ax[e] = b.Vs[i]; o.ldax[e] = proj[i].r; o.Bx[e] = proj[i].A; o.ldbx[e] = proj[i].d_in; o.Kx[e] = proj[i].r;
          ++e;
        }
        o.n_extra = e;
      }
    }
    TL_TRY(tc_gemm_grouped(probs, np, 256, status, st, use_pairs()));
    // masked rank-r terms: read-modify-write passes; those aimed at the same buffer go in successive launches
    for (int round = 0; round <= max_rank; ++round) {
      np = 0;
      for (int i = 0; i < n; ++i)
        if (dX && dX[i] && b.drop[i].xd && rank_in_set[i] == round)
          probs[np++] = prob_dX_dropout_term(proj + i, T, b.Vs[i], dX[i], b.drop[i]);
      if (np) TL_TRY(tc_gemm_grouped(probs, np, 256, status, st, 0));
    }
    return TEMPLORA_OK;
  };
  TL_TRY(launch_grads());
  TL_TRY(launch_main());
  return TEMPLORA_OK;
}

// One epoch = the chunk's T rows in slices of `batch` rows (the last may be shorter), one optimizer
// step after each slice: epochs * ceil(T / batch) steps in all.
templora_status_t update_impl(const templora_linear_t *proj, const templora_param_t *As, const templora_param_t *Bs,
                              int n_proj, int T_chunk, int batch, const void *const *x_chunk,
                              const void *const *dY_chunk, void *const *y_chunk, void *const *dX_chunk, int epochs,
                              float lr, float b1, float b2, float eps, float wd, int64_t *step_inout, void *ws_ptr,
                              size_t ws_bytes, bool dry, size_t *need, cudaStream_t st, int64_t warmup_steps = 0) {
  const int T = (batch <= 0 || batch > T_chunk) ? T_chunk : batch;   // rows of a full slice
  bool all_tc = true;
  for (int i = 0; i < n_proj; ++i) all_tc = all_tc && use_tc(proj + i, dry);
  // workspace: the largest need of any group (groups run one after another on the stream)
  size_t max_need = kStatusBytes;
  if (all_tc) {
    for (int g0 = 0; g0 < n_proj; g0 += kGroup) {
      WsAlloc m(nullptr, 0);
      GroupBufs gb;
      carve_group(proj + g0, (n_proj - g0 < kGroup) ? n_proj - g0 : kGroup, T, m, gb);
      if (m.off > max_need) max_need = m.off;
    }
  } else {
    for (int i = 0; i < n_proj; ++i) {
      WsAlloc m(nullptr, 0);
      fwd_impl(proj + i, T, nullptr, nullptr, nullptr, m, true, st);
      if (m.off > max_need) max_need = m.off;
      WsAlloc m2(nullptr, 0);
      bwd_impl(proj + i, T, nullptr, nullptr, nullptr, reinterpret_cast<void *>(16), nullptr, nullptr, 0, m2, true, st);
      if (m2.off > max_need) max_need = m2.off;
    }
  }
  if (need) *need = max_need;
  if (dry) return TEMPLORA_OK;
  if (ws_bytes < max_need) return TEMPLORA_ERR_WORKSPACE;

  std::vector<templora_param_t> all;
  all.reserve(2 * (size_t)n_proj);
  for (int i = 0; i < n_proj; ++i) { all.push_back(As[i]); all.push_back(Bs[i]); }
  const int work_bf16 = proj[0].dtype == TEMPLORA_BF16;
  const size_t esize = work_bf16 ? 2 : 4;
  std::vector<const void *> xs(n_proj), dYs(n_proj);
  std::vector<void *> ys(n_proj), dXs(n_proj);
  int64_t step = *step_inout;
  for (int e = 0; e < epochs; ++e)
   for (int r0 = 0; r0 < T_chunk; r0 += T) {
    const int rows = (T_chunk - r0 < T) ? T_chunk - r0 : T;
    for (int i = 0; i < n_proj; ++i) {
      const size_t oi = (size_t)r0 * proj[i].d_in * esize, oo = (size_t)r0 * proj[i].d_out * esize;
      xs[i] = reinterpret_cast<const uint8_t *>(x_chunk[i]) + oi;
      dYs[i] = reinterpret_cast<const uint8_t *>(dY_chunk[i]) + oo;
      ys[i] = reinterpret_cast<uint8_t *>(y_chunk[i]) + oo;
      dXs[i] = (dX_chunk && dX_chunk[i]) ? reinterpret_cast<uint8_t *>(dX_chunk[i]) + oi : nullptr;
    }
    const void *const *x = xs.data();
    const void *const *dY = dYs.data();
    void *const *y = ys.data();
    void *const *dX = dX_chunk ? dXs.data() : nullptr;
    if (all_tc) {
      for (int g0 = 0; g0 < n_proj; g0 += kGroup) {
        const int n = (n_proj - g0 < kGroup) ? n_proj - g0 : kGroup;
        WsAlloc a(ws_ptr, ws_bytes);
        GroupBufs gb;
        carve_group(proj + g0, n, rows, a, gb);
        if (a.overflow) return TEMPLORA_ERR_WORKSPACE;
        TL_TRY(update_group_tc(proj + g0, As + g0, Bs + g0, n, rows, x + g0, dY + g0, y + g0, dX ? dX + g0 : nullptr,
                               gb, a.status(), (uint64_t)step, st));
      }
    } else {
      for (int i = 0; i < n_proj; ++i) {
        templora_linear_t li = proj[i];
        li.dropout_offset += (uint64_t)step;   // a new mask for every optimizer step
        WsAlloc a(ws_ptr, ws_bytes);
        TL_TRY(fwd_impl(&li, rows, x[i], y[i], nullptr, a, false, st));
        WsAlloc c(ws_ptr, ws_bytes);
        int shared_before = 0;   // an earlier projection of this step wrote the same dX: add to it
        for (int k = i - i % kGroup; k < i && dX && dX[i] && proj[i].input_group != 0; ++k)
          shared_before += (dX[k] && proj[k].input_group == proj[i].input_group) ? 1 : 0;
        const int saved_override = t_path_override;
        if (shared_before) t_path_override = 1;   // the generic kernels can accumulate into dX
        const templora_status_t rc =
            bwd_impl(&li, rows, x[i], dY[i], nullptr, dX ? dX[i] : nullptr, const_cast<float *>(As[i].grad),
                     const_cast<float *>(Bs[i].grad), 0, c, false, st, shared_before ? 1 : 0);
        t_path_override = saved_override;
        TL_TRY(rc);
      }
    }
    ++step;
    TL_TRY(adamw_launch(all.data(), (int)all.size(), templora_lr_at_step(lr, step, warmup_steps), b1, b2, eps, wd, step,
                        work_bf16, st));
    *step_inout = step;
  }
  return TEMPLORA_OK;
}


// ---------------------------------------------------------------- the MLP of a decoder block in one call
// gate = x Wg^T + s (x Ag^T) Bg^T,  up likewise,  h = SiLU(gate) * up,  y = h Wd^T + s (h Ad^T) Bd^T;
// backward from dY through down, the gating and gate/up to dX (the gradient with respect to x, the sum of the
// gate and up branches) and the six LoRA gradients; AdamW on all six.  proj = {gate, up, down}.
// On the tensor-core path with CTA pairs the gating runs in the epilogues of the frozen-weight GEMMs: gate and up
// are ONE problem whose tiles hold 128 columns of each and whose epilogue writes gate, up and h; the down
// projection's input gradient dh is never stored, its epilogue writes dgate and dup.
templora_status_t mlp_impl(const templora_linear_t *proj, const templora_param_t *As, const templora_param_t *Bs, int T,
                           const void *x, const void *dY, void *gate, void *up, void *h, void *y, void *dX, int epochs,
                           float lr, float b1, float b2, float eps, float wd, int64_t *step_inout, void *ws_ptr,
                           size_t ws_bytes, bool dry, size_t *need, cudaStream_t st) {
  const templora_linear_t *lg = proj, *lu = proj + 1, *ld = proj + 2;
  const int d_ff = lg->d_out;
  const size_t esize = lg->dtype == TEMPLORA_BF16 ? 2 : 4;
  const bool all_tc = use_tc(lg, dry) && use_tc(lu, dry) && use_tc(ld, dry);
  const bool fused = all_tc && use_pairs() && lg->r == lu->r;
  const int work_bf16 = lg->dtype == TEMPLORA_BF16;
  std::vector<templora_param_t> all;
  if (!dry)
    for (int i = 0; i < 3; ++i) { all.push_back(As[i]); all.push_back(Bs[i]); }
  int64_t step = dry ? 0 : *step_inout;

  if (all_tc) {
    WsAlloc a(dry ? nullptr : ws_ptr, ws_bytes);
    GroupBufs b;
    carve_group(proj, 3, T, a, b);
    __nv_bfloat16 *dgate = a.take<__nv_bfloat16>((size_t)T * d_ff);
    __nv_bfloat16 *dup = a.take<__nv_bfloat16>((size_t)T * d_ff);
    __nv_bfloat16 *dh = a.take<__nv_bfloat16>((size_t)T * d_ff);   // used only when the gating is not fused
    if (need) *need = a.off;
    if (dry) return TEMPLORA_OK;
    if (a.overflow) return TEMPLORA_ERR_WORKSPACE;
    DeviceStatus *status = a.status();
    auto reduce_uv = [&](int i, bool u, bool v) -> templora_status_t {
      ReduceJob jobs[2];
      int nj = 0;
      const long long Tr = (long long)T * proj[i].r;
      if (u) jobs[nj++] = ReduceJob{b.Upart[i], b.su[i], Tr, Tr, proj[i].s, 1.f, nullptr, 0, b.Us[i]};
      if (v) jobs[nj++] = ReduceJob{b.Vpart[i], b.sv[i], Tr, Tr, proj[i].s, 1.f, nullptr, 0, b.Vs[i]};
      return reduce_partials_batch(jobs, nj, st);
    };
    auto grads = [&](const int *which, int n, const void *const *xin, const void *const *dyin) -> templora_status_t {
      TcProblem probs[4];
      ReduceJob jobs[4];
      int np = 0, nj = 0;
      for (int k = 0; k < n; ++k) {
        const int i = which[k];
        const templora_linear_t *l = proj + i;
        float *gB = const_cast<float *>(Bs[i].grad), *gA = const_cast<float *>(As[i].grad);
        probs[np++] = prob_dB(l, T, dyin[k], b.Us[i], b.sb[i] > 1 ? b.dBpart[i] : gB, b.sb[i]);
        probs[np++] = prob_dA(l, T, xin[k], b.Vs[i], b.sa[i] > 1 ? b.dApart[i] : gA, b.sa[i]);
        const long long nb = (long long)l->d_out * l->r, na = (long long)l->d_in * l->r;
        if (b.sb[i] > 1) jobs[nj++] = ReduceJob{b.dBpart[i], b.sb[i], nb, nb, 1.f, 1.f, gB, 0, nullptr};
        if (b.sa[i] > 1) jobs[nj++] = ReduceJob{b.dApart[i], b.sa[i], na, na, 1.f, 1.f, gA, 0, nullptr};
      }
      TL_TRY(tc_gemm_grouped(probs, np, 64, status, st));
      if (nj) TL_TRY(reduce_partials_batch(jobs, nj, st));
      return TEMPLORA_OK;
    };
    for (int e = 0; e < epochs; ++e) {
      // forward: U of gate and up, then gate | up | h in one launch
      TcProblem sk[2] = {prob_U(lg, T, x, b.Upart[0], b.su[0]), prob_U(lu, T, x, b.Upart[1], b.su[1])};
      TL_TRY(tc_gemm_grouped(sk, 2, 64, status, st));
      {
        const long long Tr0 = (long long)T * lg->r, Tr1 = (long long)T * lu->r;
        ReduceJob jobs[2] = {ReduceJob{b.Upart[0], b.su[0], Tr0, Tr0, lg->s, 1.f, nullptr, 0, b.Us[0]},
                             ReduceJob{b.Upart[1], b.su[1], Tr1, Tr1, lu->s, 1.f, nullptr, 0, b.Us[1]}};
        TL_TRY(reduce_partials_batch(jobs, 2, st));
      }
      if (fused) {
        TcProblem p = prob_y(lg, T, x, b.Us[0], gate);
        p.epi_mode = 1;
        p.B1 = lu->W0; p.ldb1 = lu->d_in;
        p.Bext1 = lu->B; p.ldbext1 = lu->r;
        p.Aext1 = b.Us[1]; p.ldaext1 = lu->r;
        p.out1 = up; p.out2 = h;
        TL_TRY(tc_gemm_grouped(&p, 1, 256, status, st, 1));
      } else {
        TcProblem p[2] = {prob_y(lg, T, x, b.Us[0], gate), prob_y(lu, T, x, b.Us[1], up)};
        TL_TRY(tc_gemm_grouped(p, 2, 256, status, st, use_pairs()));
        TL_TRY(templora_swiglu_fwd((int64_t)T * d_ff, lg->dtype, gate, up, h, st));
      }
      // down: U from h, V from dY; its LoRA gradients; y and the gradient with respect to h
      sk[0] = prob_U(ld, T, h, b.Upart[2], b.su[2]);
      sk[1] = prob_V(ld, T, dY, b.Vpart[2], b.sv[2]);
      TL_TRY(tc_gemm_grouped(sk, 2, 64, status, st));
      TL_TRY(reduce_uv(2, true, true));
      {
        const int which[1] = {2};
        const void *xin[1] = {h}, *dyin[1] = {dY};
        TL_TRY(grads(which, 1, xin, dyin));
      }
      {
        TcProblem p[2] = {prob_y(ld, T, h, b.Us[2], y), prob_dX(ld, T, dY, b.Vs[2], fused ? dgate : dh)};
        if (fused) {
          p[1].epi_mode = 2;
          p[1].out1 = dup;
          p[1].epi_in0 = gate; p[1].epi_in1 = up;
        }
        TL_TRY(tc_gemm_grouped(p, 2, 256, status, st, use_pairs()));
        if (!fused) TL_TRY(templora_swiglu_bwd((int64_t)T * d_ff, lg->dtype, gate, up, dh, dgate, dup, st));
      }
      // gate and up backward: V, the LoRA gradients, and one summed input gradient
      sk[0] = prob_V(lg, T, dgate, b.Vpart[0], b.sv[0]);
      sk[1] = prob_V(lu, T, dup, b.Vpart[1], b.sv[1]);
      TL_TRY(tc_gemm_grouped(sk, 2, 64, status, st));
      {
        const long long Tr0 = (long long)T * lg->r, Tr1 = (long long)T * lu->r;
        ReduceJob jobs[2] = {ReduceJob{b.Vpart[0], b.sv[0], Tr0, Tr0, lg->s, 1.f, nullptr, 0, b.Vs[0]},
                             ReduceJob{b.Vpart[1], b.sv[1], Tr1, Tr1, lu->s, 1.f, nullptr, 0, b.Vs[1]}};
        TL_TRY(reduce_partials_batch(jobs, 2, st));
      }
      {
        const int which[2] = {0, 1};
        const void *xin[2] = {x, x}, *dyin[2] = {dgate, dup};
        TL_TRY(grads(which, 2, xin, dyin));
      }
      if (dX) {
        TcProblem p = prob_dX(lg, T, dgate, b.Vs[0], dX);
        p.n_extra = 2;
        p.Ax[0] = dup; p.ldax[0] = d_ff; p.Bx[0] = lu->W0; p.ldbx[0] = lu->d_in; p.Kx[0] = d_ff;
        p.Ax[1] = b.Vs[1]; p.ldax[1] = lu->r; p.Bx[1] = lu->A; p.ldbx[1] = lu->d_in; p.Kx[1] = lu->r;
        TL_TRY(tc_gemm_grouped(&p, 1, 256, status, st, use_pairs()));
      }
      ++step;
      TL_TRY(adamw_launch(all.data(), 6, lr, b1, b2, eps, wd, step, work_bf16, st));
      *step_inout = step;
    }
    return TEMPLORA_OK;
  }

  // generic kernels: the same chain from the single-projection pieces
  const int saved_override = t_path_override;
  t_path_override = 1;
  auto restore = [&](templora_status_t rc) { t_path_override = saved_override; return rc; };
  WsAlloc a(dry ? nullptr : ws_ptr, ws_bytes);
  uint8_t *dgate = a.take<uint8_t>((size_t)T * d_ff * esize);
  uint8_t *dup = a.take<uint8_t>((size_t)T * d_ff * esize);
  uint8_t *dh = a.take<uint8_t>((size_t)T * d_ff * esize);
  size_t max_need = a.off;
  for (int i = 0; i < 3; ++i) {
    WsAlloc m = a, m2 = a;
    fwd_impl(proj + i, T, nullptr, nullptr, nullptr, m, true, st);
    bwd_impl(proj + i, T, nullptr, nullptr, nullptr, reinterpret_cast<void *>(16), nullptr, nullptr, 0, m2, true, st, 1);
    if (m.off > max_need) max_need = m.off;
    if (m2.off > max_need) max_need = m2.off;
  }
  if (need) *need = max_need;
  if (dry) return restore(TEMPLORA_OK);
  if (ws_bytes < max_need) return restore(TEMPLORA_ERR_WORKSPACE);
  for (int e = 0; e < epochs; ++e) {
    auto run = [&]() -> templora_status_t {
      { WsAlloc c = a; TL_TRY(fwd_impl(lg, T, x, gate, nullptr, c, false, st)); }
      { WsAlloc c = a; TL_TRY(fwd_impl(lu, T, x, up, nullptr, c, false, st)); }
      TL_TRY(templora_swiglu_fwd((int64_t)T * d_ff, lg->dtype, gate, up, h, st));
      { WsAlloc c = a; TL_TRY(fwd_impl(ld, T, h, y, nullptr, c, false, st)); }
      { WsAlloc c = a; TL_TRY(bwd_impl(ld, T, h, dY, nullptr, dh, const_cast<float *>(As[2].grad), const_cast<float *>(Bs[2].grad), 0, c, false, st)); }
      TL_TRY(templora_swiglu_bwd((int64_t)T * d_ff, lg->dtype, gate, up, dh, dgate, dup, st));
      { WsAlloc c = a; TL_TRY(bwd_impl(lg, T, x, dgate, nullptr, dX, const_cast<float *>(As[0].grad), const_cast<float *>(Bs[0].grad), 0, c, false, st)); }
      { WsAlloc c = a; TL_TRY(bwd_impl(lu, T, x, dup, nullptr, dX, const_cast<float *>(As[1].grad), const_cast<float *>(Bs[1].grad), 0, c, false, st, dX ? 1 : 0)); }
      return TEMPLORA_OK;
    };
    const templora_status_t rc = run();
    if (rc != TEMPLORA_OK) return restore(rc);
    ++step;
    const templora_status_t ra = adamw_launch(all.data(), 6, lr, b1, b2, eps, wd, step, work_bf16, st);
    if (ra != TEMPLORA_OK) return restore(ra);
    *step_inout = step;
  }
  return restore(TEMPLORA_OK);
}

}  // namespace

// Workspace bytes that templora_decode_fwd alone needs for n tokens (0 on an invalid projection);
// holds for either kernel path.
size_t decode_workspace_need(const templora_linear_t *lin, int n) {
  if (check_linear(lin) != TEMPLORA_OK || n < 1 || n > 16) return 0;
  size_t need = kStatusBytes;
  for (int mode = 0; mode < 2; ++mode) {
    t_path_override = mode;
    WsAlloc c(nullptr, 0);
    decode_impl(lin, n, nullptr, nullptr, c, true, nullptr);
    if (c.off > need) need = c.off;
  }
  t_path_override = -1;
  return need;
}

templora_status_t decode_check_args(const templora_linear_t *lin, int n_tokens, const void *x, const void *y) {
  TL_TRY(check_linear(lin));
  TL_TRY(check_linear_ptrs(lin));
  if (n_tokens < 1 || n_tokens > 16) return TEMPLORA_ERR_INVALID_ARG;
  if (!x || !y || !aligned16(x) || !aligned16(y)) return TEMPLORA_ERR_INVALID_ARG;
  return TEMPLORA_OK;
}

}  // namespace templora

using namespace templora;

extern "C" {

size_t templora_workspace_bytes(const templora_linear_t *lin, int32_t T) {
  if (check_linear(lin) != TEMPLORA_OK || T <= 0) return 0;
  size_t need = kStatusBytes;
  cudaStream_t st = nullptr;
  // measure both kernel paths so that the figure holds whichever is selected later
  for (int mode = 0; mode < 2; ++mode) {
    t_path_override = mode;
    WsAlloc a(nullptr, 0);
    fwd_impl(lin, T, nullptr, nullptr, nullptr, a, true, st);
    if (a.off > need) need = a.off;
    WsAlloc b(nullptr, 0);
    bwd_impl(lin, T, nullptr, nullptr, nullptr, reinterpret_cast<void *>(16), nullptr, nullptr, 1, b, true, st);
    if (b.off > need) need = b.off;
    WsAlloc c(nullptr, 0);
    decode_impl(lin, T < 16 ? T : 16, nullptr, nullptr, c, true, st);
    if (c.off > need) need = c.off;
  }
  t_path_override = -1;
  return need;
}

size_t templora_update_block_workspace_bytes(const templora_linear_t *proj, int32_t n_proj, int32_t T) {
  if (!proj || n_proj <= 0 || T <= 0) return 0;
  for (int i = 0; i < n_proj; ++i)
    if (check_linear(proj + i) != TEMPLORA_OK) return 0;
  size_t need = 0, best = kStatusBytes;
  for (int mode = 0; mode < 2; ++mode) {
    t_path_override = mode;
    update_impl(proj, nullptr, nullptr, n_proj, T, T, nullptr, nullptr, nullptr, nullptr, 0, 0, 0, 0, 0, 0, nullptr,
                nullptr, 0, true, &need, nullptr);
    if (need > best) best = need;
  }
  t_path_override = -1;
  return best;
}

templora_status_t templora_linear_fwd(const templora_linear_t *lin, int32_t T, const void *x, void *y, float *U_save,
                                      void *ws, size_t ws_bytes, void *stream) {
  TL_TRY(check_linear(lin));
  TL_TRY(check_linear_ptrs(lin));
  if (T <= 0 || !x || !y || !aligned16(x) || !aligned16(y) || (U_save && !aligned16(U_save))) return TEMPLORA_ERR_INVALID_ARG;
  TL_TRY(check_ws(ws, ws_bytes));
  WsAlloc a(ws, ws_bytes);
  return fwd_impl(lin, T, x, y, U_save, a, false, reinterpret_cast<cudaStream_t>(stream));
}

templora_status_t templora_linear_bwd(const templora_linear_t *lin, int32_t T, const void *x, const void *dY,
                                      const float *U_saved, void *dX, float *dA, float *dB, int32_t accumulate,
                                      void *ws, size_t ws_bytes, void *stream) {
  TL_TRY(check_linear(lin));
  TL_TRY(check_linear_ptrs(lin));
  if (T <= 0 || !x || !dY || !dA || !dB) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(dY) || !aligned16(dA) || !aligned16(dB) || (dX && !aligned16(dX)) ||
      (U_saved && !aligned16(U_saved)))
    return TEMPLORA_ERR_INVALID_ARG;
  TL_TRY(check_ws(ws, ws_bytes));
  WsAlloc a(ws, ws_bytes);
  return bwd_impl(lin, T, x, dY, U_saved, dX, dA, dB, accumulate ? 1 : 0, a, false, reinterpret_cast<cudaStream_t>(stream));
}

templora_status_t templora_adamw_step(const templora_param_t *params, int32_t n_params, float lr, float beta1,
                                      float beta2, float eps, float weight_decay, int64_t step, int32_t work_dtype,
                                      void *stream) {
  if (!params || n_params <= 0 || step < 1) return TEMPLORA_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f) || !(lr == lr)) return TEMPLORA_ERR_INVALID_ARG;
  if (work_dtype != TEMPLORA_F32 && work_dtype != TEMPLORA_BF16) return TEMPLORA_ERR_UNSUPPORTED;
  for (int i = 0; i < n_params; ++i) {
    const templora_param_t &p = params[i];
    if (p.n <= 0 || !p.master || !p.m || !p.v || !p.grad) return TEMPLORA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(p.master) | reinterpret_cast<uintptr_t>(p.m) | reinterpret_cast<uintptr_t>(p.v) |
         reinterpret_cast<uintptr_t>(p.grad)) & 3)
      return TEMPLORA_ERR_INVALID_ARG;
  }
  return adamw_launch(params, n_params, lr, beta1, beta2, eps, weight_decay, step, work_dtype == TEMPLORA_BF16,
                      reinterpret_cast<cudaStream_t>(stream));
}

templora_status_t templora_decode_fwd(const templora_linear_t *lin, int32_t n_tokens, const void *x, void *y, void *ws,
                                      size_t ws_bytes, void *stream) {
  TL_TRY(decode_check_args(lin, n_tokens, x, y));
  TL_TRY(check_ws(ws, ws_bytes));
  WsAlloc a(ws, ws_bytes);
  return decode_impl(lin, n_tokens, x, y, a, false, reinterpret_cast<cudaStream_t>(stream));
}

size_t templora_decode_block_workspace_bytes(const templora_linear_t *proj, int32_t n_proj) {
  if (!proj || n_proj <= 0) return 0;
  for (int i = 0; i < n_proj; ++i)
    if (check_linear(proj + i) != TEMPLORA_OK) return 0;
  size_t need = 0, best = kStatusBytes;
  for (int mode = 0; mode < 2; ++mode) {
    t_path_override = mode;
    decode_block_impl(proj, n_proj, 16, nullptr, nullptr, nullptr, 0, true, &need, nullptr);
    if (need > best) best = need;
  }
  t_path_override = -1;
  return best;
}

templora_status_t templora_decode_block_fwd(const templora_linear_t *proj, int32_t n_proj, int32_t n_tokens,
                                            const void *const *x, void *const *y, void *ws, size_t ws_bytes,
                                            void *stream) {
  if (!proj || n_proj <= 0 || !x || !y || n_tokens < 1 || n_tokens > 16) return TEMPLORA_ERR_INVALID_ARG;
  for (int i = 0; i < n_proj; ++i) {
    TL_TRY(check_linear(proj + i));
    TL_TRY(check_linear_ptrs(proj + i));
    if (!x[i] || !y[i] || !aligned16(x[i]) || !aligned16(y[i])) return TEMPLORA_ERR_INVALID_ARG;
  }
  TL_TRY(check_ws(ws, ws_bytes));
  size_t need = 0;
  decode_block_impl(proj, n_proj, n_tokens, nullptr, nullptr, nullptr, 0, true, &need, nullptr);
  if (ws_bytes < need) return TEMPLORA_ERR_WORKSPACE;
  return decode_block_impl(proj, n_proj, n_tokens, x, y, ws, ws_bytes, false, nullptr,
                           reinterpret_cast<cudaStream_t>(stream));
}

templora_status_t templora_update_block(const templora_linear_t *proj, const templora_param_t *A_state,
                                        const templora_param_t *B_state, int32_t n_proj, int32_t T,
                                        const void *const *x, const void *const *dY, void *const *y, void *const *dX,
                                        int32_t epochs, float lr, float beta1, float beta2, float eps,
                                        float weight_decay, int64_t *step_inout, void *ws, size_t ws_bytes,
                                        void *stream) {
  return templora_update_block_batched(proj, A_state, B_state, n_proj, T, T, x, dY, y, dX, epochs, lr, beta1, beta2, eps,
                                       weight_decay, step_inout, ws, ws_bytes, stream);
}

float templora_lr_at_step(float lr, int64_t step, int64_t warmup_steps) {
  if (warmup_steps <= 0 || step >= warmup_steps) return lr;
  if (step < 0) step = 0;
  return (float)((double)lr * ((double)step / (double)warmup_steps));
}

templora_status_t templora_update_block_batched(const templora_linear_t *proj, const templora_param_t *A_state,
                                                const templora_param_t *B_state, int32_t n_proj, int32_t T,
                                                int32_t batch_tokens, const void *const *x, const void *const *dY,
                                                void *const *y, void *const *dX, int32_t epochs, float lr,
                                                float beta1, float beta2, float eps, float weight_decay,
                                                int64_t *step_inout, void *ws, size_t ws_bytes, void *stream) {
  return templora_update_block_warmup(proj, A_state, B_state, n_proj, T, batch_tokens, x, dY, y, dX, epochs, lr, 0, beta1,
                                      beta2, eps, weight_decay, step_inout, ws, ws_bytes, stream);
}

templora_status_t templora_update_block_warmup(const templora_linear_t *proj, const templora_param_t *A_state,
                                               const templora_param_t *B_state, int32_t n_proj, int32_t T,
                                               int32_t batch_tokens, const void *const *x, const void *const *dY,
                                               void *const *y, void *const *dX, int32_t epochs, float lr,
                                               int64_t warmup_steps, float beta1, float beta2, float eps,
                                               float weight_decay, int64_t *step_inout, void *ws, size_t ws_bytes,
                                               void *stream) {
  if (batch_tokens < 1 || warmup_steps < 0) return TEMPLORA_ERR_INVALID_ARG;
  if (!proj || !A_state || !B_state || n_proj <= 0 || T <= 0 || !x || !dY || !y || epochs < 0 || !step_inout ||
      *step_inout < 0)
    return TEMPLORA_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f)) return TEMPLORA_ERR_INVALID_ARG;
  for (int i = 0; i < n_proj; ++i) {
    TL_TRY(check_linear(proj + i));
    TL_TRY(check_linear_ptrs(proj + i));
    if (proj[i].dtype != proj[0].dtype) return TEMPLORA_ERR_UNSUPPORTED;
    if (!x[i] || !dY[i] || !y[i] || !aligned16(x[i]) || !aligned16(dY[i]) || !aligned16(y[i])) return TEMPLORA_ERR_INVALID_ARG;
    if (dX && dX[i] && !aligned16(dX[i])) return TEMPLORA_ERR_INVALID_ARG;
    if (proj[i].input_group != 0 && dX && dX[i]) {
      // members of an input group (within one run of eight projections): one dX buffer, one input width, at most three
      int sharers = 0;
      for (int k = i - i % kGroup; k < i; ++k)
        if (dX[k] && proj[k].input_group == proj[i].input_group) {
          ++sharers;
          if (proj[k].d_in != proj[i].d_in || dX[k] != dX[i]) return TEMPLORA_ERR_INVALID_ARG;
        }
      if (sharers > 2) return TEMPLORA_ERR_INVALID_ARG;
    }
    const templora_param_t &a = A_state[i], &b = B_state[i];
    if (a.n != (int64_t)proj[i].r * proj[i].d_in || b.n != (int64_t)proj[i].d_out * proj[i].r) return TEMPLORA_ERR_INVALID_ARG;
    if (!a.master || !a.m || !a.v || !a.grad || !b.master || !b.m || !b.v || !b.grad) return TEMPLORA_ERR_INVALID_ARG;
    if (!aligned16(a.grad) || !aligned16(b.grad)) return TEMPLORA_ERR_INVALID_ARG;
    // the projections must read what the optimizer writes
    const void *wa = proj[i].dtype == TEMPLORA_BF16 ? a.work : (const void *)a.master;
    const void *wb = proj[i].dtype == TEMPLORA_BF16 ? b.work : (const void *)b.master;
    if (proj[i].A != wa || proj[i].B != wb) return TEMPLORA_ERR_INVALID_ARG;
  }
  TL_TRY(check_ws(ws, ws_bytes));
  return update_impl(proj, A_state, B_state, n_proj, T, batch_tokens, x, dY, y, dX, epochs, lr, beta1, beta2, eps,
                     weight_decay, step_inout, ws, ws_bytes, false, nullptr, reinterpret_cast<cudaStream_t>(stream),
                     warmup_steps);
}

static templora_status_t check_mlp(const templora_linear_t *proj) {
  if (!proj) return TEMPLORA_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i) {
    TL_TRY(check_linear(proj + i));
    if (proj[i].dtype != proj[0].dtype) return TEMPLORA_ERR_UNSUPPORTED;
    if (proj[i].dropout_p != 0.f) return TEMPLORA_ERR_UNSUPPORTED;
  }
  // gate and up read the same input and feed the gating; down reads its result
  if (proj[0].d_in != proj[1].d_in || proj[0].d_out != proj[1].d_out || proj[2].d_in != proj[0].d_out)
    return TEMPLORA_ERR_INVALID_ARG;
  return TEMPLORA_OK;
}

size_t templora_update_mlp_workspace_bytes(const templora_linear_t *proj, int32_t T) {
  if (check_mlp(proj) != TEMPLORA_OK || T <= 0) return 0;
  size_t need = 0, best = kStatusBytes;
  for (int mode = 0; mode < 2; ++mode) {
    t_path_override = mode;
    mlp_impl(proj, nullptr, nullptr, T, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, 0, 0, 0, 0, 0,
             nullptr, nullptr, 0, true, &need, nullptr);
    if (need > best) best = need;
  }
  t_path_override = -1;
  return best;
}

templora_status_t templora_update_mlp(const templora_linear_t *proj, const templora_param_t *A_state,
                                      const templora_param_t *B_state, int32_t T, const void *x, const void *dY,
                                      void *gate, void *up, void *h, void *y, void *dX, int32_t epochs, float lr,
                                      float beta1, float beta2, float eps, float weight_decay, int64_t *step_inout,
                                      void *ws, size_t ws_bytes, void *stream) {
  TL_TRY(check_mlp(proj));
  if (!A_state || !B_state || T <= 0 || !x || !dY || !gate || !up || !h || !y || epochs < 0 || !step_inout || *step_inout < 0)
    return TEMPLORA_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f)) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(dY) || !aligned16(gate) || !aligned16(up) || !aligned16(h) || !aligned16(y) ||
      (dX && !aligned16(dX)))
    return TEMPLORA_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i) {
    TL_TRY(check_linear_ptrs(proj + i));
    const templora_param_t &a = A_state[i], &b = B_state[i];
    if (a.n != (int64_t)proj[i].r * proj[i].d_in || b.n != (int64_t)proj[i].d_out * proj[i].r) return TEMPLORA_ERR_INVALID_ARG;
    if (!a.master || !a.m || !a.v || !a.grad || !b.master || !b.m || !b.v || !b.grad) return TEMPLORA_ERR_INVALID_ARG;
    if (!aligned16(a.grad) || !aligned16(b.grad)) return TEMPLORA_ERR_INVALID_ARG;
    const void *wa = proj[i].dtype == TEMPLORA_BF16 ? a.work : (const void *)a.master;
    const void *wb = proj[i].dtype == TEMPLORA_BF16 ? b.work : (const void *)b.master;
    if (proj[i].A != wa || proj[i].B != wb) return TEMPLORA_ERR_INVALID_ARG;
  }
  TL_TRY(check_ws(ws, ws_bytes));
  size_t need = 0;
  mlp_impl(proj, nullptr, nullptr, T, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, 0, 0, 0, 0, 0, nullptr,
           nullptr, 0, true, &need, nullptr);
  if (ws_bytes < need) return TEMPLORA_ERR_WORKSPACE;
  return mlp_impl(proj, A_state, B_state, T, x, dY, gate, up, h, y, dX, epochs, lr, beta1, beta2, eps, weight_decay,
                  step_inout, ws, ws_bytes, false, nullptr, reinterpret_cast<cudaStream_t>(stream));
}

templora_status_t templora_update_attn_in(const templora_linear_t *proj, const templora_param_t *A_state,
                                          const templora_param_t *B_state, int32_t n_proj, int32_t T, const void *x,
                                          const void *norm_weight, float norm_eps, const void *const *dY, void *xn,
                                          void *const *y, void *dXn, void *dX, int32_t epochs, float lr, float beta1,
                                          float beta2, float eps, float weight_decay, int64_t *step_inout, void *ws,
                                          size_t ws_bytes, void *stream) {
  if (!proj || n_proj < 1 || n_proj > 3 || T <= 0 || !x || !norm_weight || !dY || !xn || !y || !dXn) return TEMPLORA_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(norm_weight) || !aligned16(xn) || !aligned16(dXn) || (dX && !aligned16(dX)))
    return TEMPLORA_ERR_INVALID_ARG;
  if (!(norm_eps >= 0.f)) return TEMPLORA_ERR_INVALID_ARG;
  // the projections read ONE tensor (the normalised input) and their input gradients are summed into ONE buffer
  templora_linear_t shared[3];
  const void *xs[3];
  void *dXs[3];
  for (int i = 0; i < n_proj; ++i) {
    TL_TRY(check_linear(proj + i));
    if (proj[i].d_in != proj[0].d_in || proj[i].dtype != proj[0].dtype) return TEMPLORA_ERR_INVALID_ARG;
    shared[i] = proj[i];
    shared[i].input_group = 1;
    xs[i] = xn;
    dXs[i] = dXn;
  }
  const int d = proj[0].d_in, dt = proj[0].dtype;
  // every argument check of the update runs before anything is enqueued (zero epochs: checks only)
  {
    int64_t probe = step_inout ? *step_inout : 0;
    TL_TRY(templora_update_block(shared, A_state, B_state, n_proj, T, xs, dY, y, dXs, 0, lr, beta1, beta2, eps,
                                 weight_decay, step_inout ? &probe : nullptr, ws, ws_bytes, stream));
    if (epochs < 0) return TEMPLORA_ERR_INVALID_ARG;
  }
  TL_TRY(templora_rmsnorm_fwd(T, d, dt, x, norm_weight, norm_eps, xn, stream));
  TL_TRY(templora_update_block(shared, A_state, B_state, n_proj, T, xs, dY, y, dXs, epochs, lr, beta1, beta2, eps,
                               weight_decay, step_inout, ws, ws_bytes, stream));
  if (dX && epochs > 0) TL_TRY(templora_rmsnorm_bwd(T, d, dt, x, norm_weight, dXn, norm_eps, dX, stream));
  return TEMPLORA_OK;
}

const char *templora_status_string(templora_status_t st) {
  switch (st) {
    case TEMPLORA_OK: return "ok";
    case TEMPLORA_ERR_INVALID_ARG: return "invalid argument";
    case TEMPLORA_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case TEMPLORA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case TEMPLORA_ERR_CUDA: return "CUDA call failed";
    case TEMPLORA_ERR_TIMEOUT: return "bounded device-side wait expired";
  }
  return "unknown status";
}

templora_status_t templora_read_device_status(void *ws, void *stream, int32_t *code, int32_t *where) {
  if (!ws || !code || !where) return TEMPLORA_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return TEMPLORA_ERR_CUDA;
  int32_t rec[2] = {0, 0};
  if (cudaMemcpy(rec, ws, sizeof(rec), cudaMemcpyDeviceToHost) != cudaSuccess) return TEMPLORA_ERR_CUDA;
  *code = rec[0];
  *where = rec[1];
  return TEMPLORA_OK;
}

templora_status_t templora_selftest_bounded_wait(void *ws, size_t ws_bytes, int32_t limit_ms, void *stream) {
  TL_TRY(check_ws(ws, ws_bytes));
  if (limit_ms < 1 || limit_ms > 1000) return TEMPLORA_ERR_INVALID_ARG;
  return tc_wait_selftest(reinterpret_cast<DeviceStatus *>(ws), (unsigned long long)limit_ms * 1000000ull,
                          reinterpret_cast<cudaStream_t>(stream));
}

templora_status_t templora_set_stream_sm_limit(void *stream, int32_t max_sms) {
  if (max_sms < 0) return TEMPLORA_ERR_INVALID_ARG;
  tc_set_stream_sm_limit(reinterpret_cast<cudaStream_t>(stream), max_sms);
  return TEMPLORA_OK;
}

int32_t templora_set_kernel_path(int32_t mode) {
  return g_kernel_path.exchange((mode == 1 || mode == 2) ? mode : 0);
}

}  // extern "C"
