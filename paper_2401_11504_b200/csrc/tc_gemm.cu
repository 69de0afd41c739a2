// Persistent grouped GEMM on the sm_100a tensor cores (tcgen05 + TMEM accumulators, operands
// staged by TMA).  One launch runs a list of problems
//     D[M,N] = Aop[M,K] Bop[N,K]^T  (+ Aext[M,Kext] Bext[N,Kext]^T)
// with bf16 operands and fp32 accumulation.  The optional second product runs as extra
// k-blocks of the same tile loop into the same TMEM accumulator: that is how the rank-r LoRA
// term s U B^T (forward) and s V A (input gradient) are fused into the frozen-weight GEMM.
// Either operand may be stored K-contiguous or M/N-contiguous, so dY W0 (W0 row-major, contracted
// over its rows) and the token-dimension reductions dY^T U and x^T V need no transposed copies.
// Split-K partial outputs are written to separate slabs and summed later in a fixed order.
//
// CTA = 6 warps: warp 0 issues TMA loads, warp 1 owns TMEM and issues the MMAs, warps 2..5 drain
// the accumulator (TMEM -> registers -> global).  Two accumulator buffers let the epilogue of one
// tile overlap the mainloop of the next.  Every mbarrier wait is bounded: when a wait runs out the
// CTA records TEMPLORA_ERR_TIMEOUT in the device status record, drains what it has in flight,
// frees its TMEM and returns.
//
// Work items (problem, m-tile, n-tile, k-split) are drawn from a counter in the status record at the
// head of the workspace: CTA b starts with item b and then takes "next" atomically, so the tail of
// a launch is balanced whatever the mix of long and short items.  The counter must be zero at
// launch (the workspace head is zeroed once by the caller); the last CTA to finish resets it.
#include "common.cuh"
#include "tc_device.cuh"
#include "tc_host.h"

#include <cuda.h>

#include <atomic>
#include <mutex>
#include <unordered_map>

namespace templora {
namespace {

constexpr int kThreads = 192;
constexpr int kThreads2 = 224;   // single-CTA GEMM kernel: one more warp, the second TMA producer
constexpr int kSched = 4;  // depth of the work-item ring between the producer and its consumers

constexpr int kStageA = BM * BK * 2;  // 16 KB
// KPS = k-blocks per pipeline stage.  The decode stream (BN = 16) moves two k-blocks per stage so that
// the two 128-byte pieces of every W0 row are requested back to back (256 contiguous bytes per row).
template <int BN, int STAGES, int TMEM_COLS, int KPS> struct CfgBase {
  static constexpr int kStages = STAGES, kTmemCols = TMEM_COLS, kKps = KPS;
  static constexpr int kStageB = BN * BK * 2;
  static constexpr int kSub = kStageA + kStageB;       // one k-block of A and B
  static constexpr int kStage = KPS * kSub;
  static constexpr int kSmemBytes = STAGES * kStage + 1024 /*barriers*/ + 1024 /*alignment slack*/;
};
template <int BN> struct Cfg;
template <> struct Cfg<256> : CfgBase<256, 4, 512, 1> {};
#ifndef TL_C64_STAGES
#define TL_C64_STAGES 8
#endif
#ifndef TL_C64_KPS
#define TL_C64_KPS 1
#endif
#ifndef TL_C64_HINT
#define TL_C64_HINT 0
#endif
template <> struct Cfg<64> : CfgBase<64, TL_C64_STAGES, 128, TL_C64_KPS> {};
template <> struct Cfg<16> : CfgBase<16, 3, 32, 4> {};

constexpr int kMaxExtra = 4;   // further operand pairs accumulated into the same output tile
struct alignas(64) DevProb {
  CUtensorMap tmA, tmB, tmAe, tmBe;
  CUtensorMap tmXa[kMaxExtra], tmXb[kMaxExtra];
  CUtensorMap tmOut;            // CTA-pair kernel: the bf16 row-major output, boxes of 32 rows x 64 columns
  int kb_x[kMaxExtra], kb_xtot;   // k-blocks of each extra pair and their sum (the pairs follow the extension)
  long long out_s0, out_s1, out_split;
  void *out;
  int M, N, kb_main, kb_ext, splits, m_tiles, n_tiles, item_start, a_mn, b_mn, out_f32, pad;
  const uint8_t *epi_mask;      // "add under a mask" epilogue (dropout term of dX); nullptr = plain store
  long long epi_mask_pitch;
  float epi_scale;
  int pad3;
  // CTA-pair kernel, gating fused into the epilogue (TcProblem::epi_mode).  Mode 1 keeps the up projection's
  // operand maps in tmXb[1] (W_up), tmXa[0] / tmXb[0] (s*U_up, B_up: the extra pair) and the maps of its further
  // outputs in tmXa[1] (up) and tmXa[2] (h); mode 2 keeps the map of dup in tmXa[1].  Output maps of these modes
  // have boxes of 32 rows x 32 columns, not swizzled.
  const __nv_bfloat16 *epi_in0, *epi_in1;
  int epi_mode, pad4;
};
struct DevGroup {
  DevProb p[kTcMaxProblems];
  DeviceStatus *status;
  int n_prob, n_items;
};

struct Item {
  int p, m0, nt, split, kb0, kb1, next;
};


__device__ __forceinline__ Item decode_item(const DevGroup &g, int item) {
  int p = 0;
  while (p + 1 < g.n_prob && item >= g.p[p + 1].item_start) ++p;
  const DevProb &q = g.p[p];
  int local = item - q.item_start;
  Item it;
  it.p = p;
  it.m0 = (local % q.m_tiles) * BM;
  local /= q.m_tiles;
  it.nt = local % q.n_tiles;
  it.split = local / q.n_tiles;
  it.kb0 = (int)((long long)q.kb_main * it.split / q.splits);
  it.kb1 = (int)((long long)q.kb_main * (it.split + 1) / q.splits);
  it.next = (it.split == q.splits - 1) ? q.kb_ext + q.kb_xtot : 0;
  return it;
}

// Walks the k-blocks of a work item in order: the streamed range of the main operand pair, then the
// extension pair, then the extra pairs.  take() yields the maps and the k element offset of the next block.
struct KCursor {
  const DevProb &q;
  const CUtensorMap *ma, *mb;
  int seg, left, kel;
  __device__ __forceinline__ KCursor(const DevProb &q_, int kb0, int nmain)
      : q(q_), ma(&q_.tmA), mb(&q_.tmB), seg(0), left(nmain), kel(kb0 * BK) {}
  __device__ __forceinline__ void take(const CUtensorMap *&a, const CUtensorMap *&b, int &k) {
    while (left == 0 && seg <= kMaxExtra) {   // the caller never asks for more blocks than the item has
      ++seg;
      kel = 0;
      if (seg == 1) { ma = &q.tmAe; mb = &q.tmBe; left = q.kb_ext; }
      else { ma = &q.tmXa[seg - 2]; mb = &q.tmXb[seg - 2]; left = q.kb_x[seg - 2]; }
    }
    a = ma; b = mb; k = kel;
    kel += BK;
    --left;
  }
};

// ------------------------------------------------------------------ epilogue stores
template <int NV>
__device__ __forceinline__ void store_chunk(const DevProb &q, const uint32_t (&v)[32], int row, int col0, int split) {
  if (row >= q.M || col0 >= q.N) return;
  const long long base = (long long)split * q.out_split + (long long)row * q.out_s0 + (long long)col0 * q.out_s1;
  const int ncol = (q.N - col0 < NV) ? q.N - col0 : NV;
  if (q.epi_mask) {
    // out = out_old + (keep ? epi_scale * D : 0); bf16, row-major; col0 is a multiple of 8
    __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(q.out) + base;
    const uint8_t *mrow = q.epi_mask + (long long)row * q.epi_mask_pitch + (col0 >> 3);
    if (ncol == NV && ((reinterpret_cast<uintptr_t>(o) & 15) == 0)) {
      // all old values of the chunk are requested before any is used: one memory round trip per chunk
      uint4 w[NV / 8];
      uint32_t bits = 0;
#pragma unroll
      for (int c = 0; c < NV / 8; ++c) w[c] = *reinterpret_cast<const uint4 *>(o + 8 * c);
#pragma unroll
      for (int c = 0; c < NV / 8; ++c) bits |= (uint32_t)mrow[c] << (8 * c);
#pragma unroll
      for (int c = 0; c < NV / 8; ++c) {
        __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&w[c]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float2 old = __bfloat1622float2(h[e]);
          if ((bits >> (8 * c + 2 * e)) & 1) old.x += q.epi_scale * __uint_as_float(v[8 * c + 2 * e]);
          if ((bits >> (8 * c + 2 * e + 1)) & 1) old.y += q.epi_scale * __uint_as_float(v[8 * c + 2 * e + 1]);
          h[e] = __floats2bfloat162_rn(old.x, old.y);
        }
      }
#pragma unroll
      for (int c = 0; c < NV / 8; ++c) *reinterpret_cast<uint4 *>(o + 8 * c) = w[c];
    } else {
      for (int c = 0; c < ncol; ++c)
        if ((mrow[c >> 3] >> (c & 7)) & 1)
          o[c] = __float2bfloat16_rn(__bfloat162float(o[c]) + q.epi_scale * __uint_as_float(v[c]));
    }
    return;
  }
  if (q.out_f32) {
    float *o = reinterpret_cast<float *>(q.out) + base;
    if (q.out_s1 == 1 && ncol == NV && ((reinterpret_cast<uintptr_t>(o) & 15) == 0)) {
#pragma unroll
      for (int c = 0; c < NV; c += 4)
        *reinterpret_cast<float4 *>(o + c) = make_float4(__uint_as_float(v[c]), __uint_as_float(v[c + 1]),
                                                         __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
    } else {
#pragma unroll
      for (int c = 0; c < NV; ++c)
        if (c < ncol) o[(long long)c * q.out_s1] = __uint_as_float(v[c]);
    }
  } else {
    __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(q.out) + base;
    if (q.out_s1 == 1 && ncol == NV && ((reinterpret_cast<uintptr_t>(o) & 15) == 0)) {
#pragma unroll
      for (int c = 0; c < NV; c += 8) {
        uint4 w;
        __nv_bfloat162 t0 = __floats2bfloat162_rn(__uint_as_float(v[c]), __uint_as_float(v[c + 1]));
        __nv_bfloat162 t1 = __floats2bfloat162_rn(__uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
        __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(v[c + 4]), __uint_as_float(v[c + 5]));
        __nv_bfloat162 t3 = __floats2bfloat162_rn(__uint_as_float(v[c + 6]), __uint_as_float(v[c + 7]));
        w.x = *reinterpret_cast<uint32_t *>(&t0);
        w.y = *reinterpret_cast<uint32_t *>(&t1);
        w.z = *reinterpret_cast<uint32_t *>(&t2);
        w.w = *reinterpret_cast<uint32_t *>(&t3);
        *reinterpret_cast<uint4 *>(o + c) = w;
      }
    } else {
#pragma unroll
      for (int c = 0; c < NV; ++c)
        if (c < ncol) o[(long long)c * q.out_s1] = __float2bfloat16_rn(__uint_as_float(v[c]));
    }
  }
}

// Epilogue of the masked second pass of dX, one accumulator row of BN columns per thread:
//   dX[row, n0 + c] += keep(row, n0 + c) ? epi_scale * D[row, c] : 0
// The old values of chunk c+1 are requested while chunk c is combined and stored, so the global
// round trip of the read-modify-write overlaps the TMEM read and the arithmetic.
template <int BN>
__device__ __forceinline__ void masked_add_row(const DevProb &q, uint32_t t_row, int row, int n0) {
  const bool in_rows = row < q.M;
  __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(q.out) + (long long)row * q.out_s0;
  const uint8_t *mrow = q.epi_mask + (long long)row * q.epi_mask_pitch;
  const bool vec = in_rows && (q.out_s0 % 8 == 0) && ((reinterpret_cast<uintptr_t>(q.out) & 15) == 0);
  uint4 nxt[4];
  uint32_t nbits = 0;
  auto preload = [&](int col) {
    if (vec && col + 32 <= q.N) {
#pragma unroll
      for (int c = 0; c < 4; ++c) nxt[c] = *reinterpret_cast<const uint4 *>(orow + col + 8 * c);
      nbits = *reinterpret_cast<const uint32_t *>(mrow + (col >> 3));
    }
  };
  preload(n0);
  uint32_t v[32];
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 32) {
    const int col = n0 + c0;
    uint4 w[4] = {nxt[0], nxt[1], nxt[2], nxt[3]};
    const uint32_t bits = nbits;
    if (c0 + 32 < BN) preload(col + 32);
    tmem_ld32(t_row + c0, v);
    tmem_ld_wait();
    if (!in_rows || col >= q.N) continue;
    if (vec && col + 32 <= q.N) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&w[c]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float2 old = __bfloat1622float2(h[e]);
          if ((bits >> (8 * c + 2 * e)) & 1) old.x += q.epi_scale * __uint_as_float(v[8 * c + 2 * e]);
          if ((bits >> (8 * c + 2 * e + 1)) & 1) old.y += q.epi_scale * __uint_as_float(v[8 * c + 2 * e + 1]);
          h[e] = __floats2bfloat162_rn(old.x, old.y);
        }
        *reinterpret_cast<uint4 *>(orow + col + 8 * c) = w[c];
      }
    } else {
      const int ncol = (q.N - col < 32) ? q.N - col : 32;
      for (int c = 0; c < ncol; ++c)
        if ((mrow[(col + c) >> 3] >> ((col + c) & 7)) & 1)
          orow[col + c] = __float2bfloat16_rn(__bfloat162float(orow[col + c]) + q.epi_scale * __uint_as_float(v[c]));
    }
  }
}

// ------------------------------------------------------------------ the kernel
template <int BN>
__global__ void __launch_bounds__(kThreads2, 1) tc_gemm_kernel(const __grid_constant__ DevGroup g) {
  constexpr int kStages = Cfg<BN>::kStages;
  constexpr int kStage = Cfg<BN>::kStage;
  constexpr int kSub = Cfg<BN>::kSub;
  constexpr int kKps = Cfg<BN>::kKps;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_al = smem_raw + (smem0 - smem_u32(smem_raw));
  const uint32_t bar0 = smem0 + kStages * kStage;  // barriers: 8 bytes each
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 + a); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kStages + 4);
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_al + kStages * kStage + 512);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_al + kStages * kStage + 516);
  // work items are handed out dynamically: the producer draws the next item from a global counter
  // and passes it to the MMA thread and the epilogue warps through this small ring
  volatile int *sched_ring = reinterpret_cast<volatile int *>(smem_al + kStages * kStage + 528);
  auto sfull_bar = [&](int s) { return bar0 + 8u * (2 * kStages + 5 + s); };
  auto sempty_bar = [&](int s) { return bar0 + 8u * (2 * kStages + 5 + kSched + s); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 4);
    }
    mbar_init(drain_bar, 1);
    for (int s = 0; s < kSched; ++s) {
      mbar_init(sfull_bar(s), 1);
      mbar_init(sempty_bar(s), 6);  // the B-operand producer, the MMA thread, one lane of each epilogue warp
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                 "r"((uint32_t)Cfg<BN>::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_prologue();   // the set-up above touched no global memory and may overlap the previous kernel's tail

  if (warp == 0) {
    // ===================== TMA producer: hands out the items and loads the A operand =====================
    // (the B operand is loaded by warp 6: one thread issuing every copy was close to the critical path)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      int item = blockIdx.x, sslot = 0;
      uint32_t sphase = 0;
      const uint64_t stream_policy = l2_policy_evict_first();
      while (ok) {
        if (!mbar_wait(sempty_bar(sslot), sphase ^ 1u, abort_flag, g.status, 110)) { ok = false; break; }
        sched_ring[sslot] = item;
        mbar_arrive(sfull_bar(sslot));
        if (++sslot == kSched) { sslot = 0; sphase ^= 1u; }
        if (item >= g.n_items) break;  // the end marker has been passed on
        const int next_item = (int)gridDim.x + atomicAdd(&g.status->sched_next, 1);  // drawn early, used late
        const Item it = decode_item(g, item);
        const DevProb &q = g.p[it.p];
        const int pa_mn = q.a_mn;
        const int nmain = it.kb1 - it.kb0;
        const int nkb = nmain + it.next;
        KCursor cur(q, it.kb0, nmain);
        for (int i0 = 0; i0 < nkb; i0 += kKps) {
          const int cnt = (nkb - i0 < kKps) ? nkb - i0 : kKps;
          if (!mbar_wait_fast(empty_bar(stage), phase ^ 1u, abort_flag, g.status, 100)) { ok = false; break; }
          mbar_arrive_expect_tx(full_bar(stage), (uint32_t)(cnt * kSub));
          for (int j = 0; j < cnt; ++j) {
            const CUtensorMap *ma, *mb;
            int kel;
            cur.take(ma, mb, kel);
            const uint32_t sA = smem0 + stage * kStage + j * kSub;
            if (!pa_mn) {
              if constexpr (BN == 16 || (BN == 64 && TL_C64_HINT))   // decode: W0 is read exactly once; keep x, A and the split-K slabs in L2 instead
                tma_load_2d_hint(sA, ma, full_bar(stage), kel, it.m0, stream_policy);
              else
                tma_load_2d(sA, ma, full_bar(stage), kel, it.m0);
            } else {
#pragma unroll
              for (int b = 0; b < BM / 64; ++b) tma_load_2d(sA + b * 8192, ma, full_bar(stage), it.m0 + b * 64, kel);
            }
          }
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        item = next_item;
      }
      if (!ok) {
        // wait (bounded) for the copies this thread still has in flight before the CTA may exit
        long long n = issued < kStages ? issued : kStages;
        for (long long k = 0; k < n; ++k) {
          long long idx = issued - 1 - k;
          int s = (int)(idx % kStages);
          uint32_t ph = (uint32_t)((idx / kStages) & 1);
          const unsigned long long t0 = globaltimer_ns();
          while (!mbar_try(full_bar(s), ph) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 6) {
    // ===================== second TMA producer: the B operand =====================
    if (lane == 0) {
      int stage = 0, sslot = 0;
      uint32_t phase = 0, sphase = 0;
      bool ok = true;
      while (ok) {
        if (!mbar_wait(sfull_bar(sslot), sphase, abort_flag, g.status, 120)) { ok = false; break; }
        const int item = sched_ring[sslot];
        mbar_arrive(sempty_bar(sslot));
        if (++sslot == kSched) { sslot = 0; sphase ^= 1u; }
        if (item >= g.n_items) break;
        const Item it = decode_item(g, item);
        const DevProb &q = g.p[it.p];
        const int n0 = it.nt * BN;
        const int pb_mn = q.b_mn;
        const int nmain = it.kb1 - it.kb0;
        const int nkb = nmain + it.next;
        KCursor cur(q, it.kb0, nmain);
        for (int i0 = 0; i0 < nkb; i0 += kKps) {
          const int cnt = (nkb - i0 < kKps) ? nkb - i0 : kKps;
          if (!mbar_wait_fast(empty_bar(stage), phase ^ 1u, abort_flag, g.status, 121)) { ok = false; break; }
          for (int j = 0; j < cnt; ++j) {
            const CUtensorMap *ma, *mb;
            int kel;
            cur.take(ma, mb, kel);
            const uint32_t sB = smem0 + stage * kStage + j * kSub + kStageA;
            if (!pb_mn) {
              tma_load_2d(sB, mb, full_bar(stage), kel, n0);
            } else {
#pragma unroll
              for (int b = 0; b < (BN >= 64 ? BN / 64 : 1); ++b)
                tma_load_2d(sB + b * 8192, mb, full_bar(stage), n0 + b * 64, kel);
            }
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int sslot = 0;
      uint32_t sphase = 0;
      for (int local = 0; ok; ++local) {
        if (!mbar_wait(sfull_bar(sslot), sphase, abort_flag, g.status, 210)) { ok = false; break; }
        const int item = sched_ring[sslot];
        mbar_arrive(sempty_bar(sslot));
        if (++sslot == kSched) { sslot = 0; sphase ^= 1u; }
        if (item >= g.n_items) break;
        const Item it = decode_item(g, item);
        const DevProb &q = g.p[it.p];
        const int nkb = (it.kb1 - it.kb0) + it.next;
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, g.status, 200)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        const int a_mn = q.a_mn, b_mn = q.b_mn;
        const uint32_t idesc = instr_desc(BN, a_mn, b_mn);
        const uint64_t a_tmpl = smem_desc_template(a_mn), b_tmpl = smem_desc_template(b_mn);
        const uint32_t a_step = smem_desc_kstep(a_mn), b_step = smem_desc_kstep(b_mn);
        for (int i0 = 0; i0 < nkb; i0 += kKps) {
          const int cnt = (nkb - i0 < kKps) ? nkb - i0 : kKps;
          if (!mbar_wait_fast(full_bar(stage), phase, abort_flag, g.status, 201)) { ok = false; break; }
          tc_fence_after();
          for (int j = 0; j < cnt; ++j) {
            const uint32_t a_lo = (smem0 + stage * kStage + j * kSub) >> 4, b_lo = a_lo + (kStageA >> 4);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              tc_mma_bf16(d_tmem, a_tmpl | (uint64_t)(a_lo + kk * a_step), b_tmpl | (uint64_t)(b_lo + kk * b_step),
                          idesc, (i0 | j | kk) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));  // frees the smem stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(tfull_bar(acc));  // accumulator complete
      }
      if (!ok) {
        // let MMAs already issued finish before TMEM is released
        tc_commit(drain_bar);
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try(drain_bar, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else {
    // ===================== epilogue (warps 2..5) =====================
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    bool ok = true;
    int sslot = 0;
    uint32_t sphase = 0;
    for (int local = 0; ok; ++local) {
      if (!mbar_wait(sfull_bar(sslot), sphase, abort_flag, g.status, 310)) { ok = false; break; }
      const int item = sched_ring[sslot];
      __syncwarp();
      if (lane == 0) mbar_arrive(sempty_bar(sslot));
      if (++sslot == kSched) { sslot = 0; sphase ^= 1u; }
      if (item >= g.n_items) break;
      const Item it = decode_item(g, item);
      const DevProb &q = g.p[it.p];
      const int n0 = it.nt * BN;
      const int acc = local & 1;
      const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, g.status, 300)) { ok = false; break; }
      tc_fence_after();
      const int row = it.m0 + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      uint32_t v[32];
      if constexpr (BN >= 32) {
        if (q.epi_mask && BN == 256) {
          masked_add_row<BN>(q, t_row, row, n0);
        } else {
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            tmem_ld32(t_row + c0, v);
            tmem_ld_wait();
            store_chunk<32>(q, v, row, n0 + c0, it.split);
          }
        }
      } else {
        tmem_ld16(t_row, v);
        tmem_ld_wait();
        store_chunk<16>(q, v, row, n0, it.split);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg<BN>::kTmemCols)
                 : "memory");
  }
  // the last CTA to finish re-arms the item counter for the next launch on this workspace
  if (threadIdx.x == 0) {
    __threadfence();
    const int done = atomicAdd(&g.status->sched_done, 1);
    if (done == (int)gridDim.x - 1) {
      g.status->sched_next = 0;
      g.status->sched_done = 0;
      __threadfence();
    }
  }
}

// ------------------------------------------------------------------ CTA-pair kernel (256 x 256 tiles)
// Two CTAs of a cluster (one TPC) share one 256 x 256 output tile: each loads its own 128 rows of
// the A operand and its own 128-column half of the B operand, and the even CTA issues
// tcgen05.mma.cta_group::2 (M = 256), which reads both halves of B from the two CTAs' shared
// memory.  Per flop this moves 1.5x fewer operand bytes from L2 into shared memory than 128 x 256
// tiles on single CTAs, which is what bounds the frozen-weight GEMMs.  Each CTA drains its own
// 128 x 256 half of the accumulator from its own TMEM.  Items are handed out dynamically, heaviest first.
namespace pair {

constexpr int kStages = 6;
constexpr int kStageB = 128 * BK * 2;            // this CTA's half of the B tile: 16 KB
constexpr int kStage = kStageA + kStageB;        // 32 KB per CTA and stage
// Output staging: each epilogue warp converts its 32 rows x 64 columns of the accumulator to bf16 in a 4 KB
// buffer (128-byte rows, 128-byte swizzle) and hands it to a bulk tensor store, so that global memory is
// written in whole 128-byte row segments; two buffers per warp, so the next chunk is converted while the
// previous one drains.
constexpr int kRowsBeyond = 1 << 28;             // a row coordinate past any tensor: the copy delivers zeros
constexpr int kOutBox = 32 * 64 * 2;             // 4 KB
constexpr int kOutStaging = 4 * 2 * kOutBox;     // 32 KB per CTA
constexpr int kSmemBytes = kStages * kStage + kOutStaging + 1024 + 1024;
constexpr int kTmemCols = 512;                   // two 256-column accumulators
constexpr int kPairThreads = 224;                // producer (A), MMA, four epilogue warps, producer (B)

// TMA load whose completion is signalled on a barrier that may live in the peer CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster, int c0,
                                                 int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {  // arrives on `bar` in both CTAs of the pair
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ uint32_t instr_desc_pair(int a_mn, int b_mn) {  // M = 256, N = 256
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// item -> (problem, 256-row tile, 256-column tile); no split-K on this path
__device__ __forceinline__ Item decode_item_pair(const DevGroup &g, int item) {
  int p = 0;
  while (p + 1 < g.n_prob && item >= g.p[p + 1].item_start) ++p;
  const DevProb &q = g.p[p];
  int local = item - q.item_start;
  Item it;
  it.p = p;
  it.m0 = (local % q.m_tiles) * 256;
  it.nt = local / q.m_tiles;
  it.split = 0;
  it.kb0 = 0;
  it.kb1 = q.kb_main;
  it.next = q.kb_ext + q.kb_xtot;
  return it;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
    tc_gemm_pair_kernel(const __grid_constant__ DevGroup g) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_al = smem_raw + (smem0 - smem_u32(smem_raw));
  const uint32_t out_stage0 = smem0 + kStages * kStage;   // 1024-byte aligned: the swizzle pattern repeats every 1 KB
  const uint32_t bar0 = out_stage0 + kOutStaging;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };                        // used in the even CTA
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };           // one per CTA
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };       // one per CTA
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 + a); };  // used in the even CTA
  const uint32_t drain_bar = bar0 + 8u * (2 * kStages + 4);
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_al + kStages * kStage + kOutStaging + 512);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_al + kStages * kStage + kOutStaging + 516);
  // Work items are handed out dynamically: the even CTA's A-operand producer draws them from the counter in
  // the workspace head (heaviest problems come first, so this is longest-processing-time-first scheduling)
  // and writes each into the item rings of both CTAs; every other role takes its items from its CTA's ring.
  volatile int *sched_ring = reinterpret_cast<volatile int *>(smem_al + kStages * kStage + kOutStaging + 528);
  const uint32_t ring0 = bar0 + 528;
  auto sfull_bar = [&](int s) { return bar0 + 8u * (2 * kStages + 5 + s); };            // one per CTA
  auto sempty_bar = [&](int s) { return bar0 + 8u * (2 * kStages + 5 + kSched + s); };  // used in the even CTA
  // readers of a ring slot: even CTA: B producer, MMA thread, 4 epilogue warps; odd CTA: both producers, 4 epilogue warps
  constexpr int kRingReaders = 12;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();      // 0: issues the MMAs; 1: its peer
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);    // the even CTA's expect_tx covers the bytes of both CTAs
      mbar_init(empty_bar(s), 1);   // one multicast commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);   // one multicast commit
      mbar_init(tempty_bar(a), 8);  // four epilogue warps in each CTA
    }
    mbar_init(drain_bar, 1);
    for (int s = 0; s < kSched; ++s) {
      mbar_init(sfull_bar(s), 1);
      mbar_init(sempty_bar(s), kRingReaders);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the peer's barriers are initialised before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_prologue();   // the set-up above touched no global memory and may overlap the previous kernel's tail

  // take the next item from this CTA's ring and hand the slot back to the dealer
  auto ring_take = [&](int &sslot, uint32_t &sphase, int where, int &item) -> bool {
    if (!mbar_wait_acq_cluster(sfull_bar(sslot), sphase, abort_flag, g.status, where)) return false;
    item = sched_ring[sslot];
    return true;
  };
  auto ring_release = [&](int &sslot, uint32_t &sphase) {
    mbar_arrive_remote_plain(mapa_shared(sempty_bar(sslot), 0));
    if (++sslot == kSched) { sslot = 0; sphase ^= 1u; }
  };

  if (warp == 0 || warp == 6) {
    // ===================== TMA producers (both CTAs): warp 0 loads the A operand, warp 6 the B operand ==========
    // Two threads because one thread issuing every copy of a k-block was close to the critical path.
    const bool do_a = warp == 0;
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      const uint32_t full0 = mapa_shared(full_bar(0), 0);
      const bool dealer = do_a && rank == 0;
      int sslot = 0;
      uint32_t sphase = 0;
      // the dealer: write an item into both CTAs' rings (the slot must have been handed back by all its readers)
      auto deal = [&](int it) -> bool {
        if (!mbar_wait(sempty_bar(sslot), sphase ^ 1u, abort_flag, g.status, 410)) return false;
#pragma unroll
        for (int r = 0; r < 2; ++r) st_cluster_s32(mapa_shared(ring0 + 4u * sslot, (uint32_t)r), it);
#pragma unroll
        for (int r = 0; r < 2; ++r)   // release at cluster scope: the store above is visible to whoever sees this arrival
          mbar_arrive_cluster(mapa_shared(sfull_bar(sslot), (uint32_t)r));
        if (++sslot == kSched) { sslot = 0; sphase ^= 1u; }
        return true;
      };
      // it deals one item ahead and draws two ahead, so the counter's round trip is never waited for
      int item = pair_id, next_item = 0, drawn = 0;
      if (dealer) {
        next_item = n_pairs + atomicAdd(&g.status->sched_next, 1);
        ok = deal(item);
      }
      while (ok) {
        if (dealer) {
          if (item >= g.n_items) break;   // the end marker has been passed on
          if (!deal(next_item)) { ok = false; break; }
          drawn = next_item < g.n_items ? n_pairs + atomicAdd(&g.status->sched_next, 1) : next_item;
        } else {
          if (!ring_take(sslot, sphase, 411, item)) { ok = false; break; }
          ring_release(sslot, sphase);
          if (item >= g.n_items) break;
        }
        const Item it = decode_item_pair(g, item);
        const DevProb &q = g.p[it.p];
        const int m0 = it.m0 + (int)rank * 128;          // this CTA's rows of the A operand
        // this CTA's half of the B operand: 128 of the tile's 256 columns - or, for a "gate | up" problem, the
        // tile's 128 rows of this CTA's own projection (even CTA: gate, odd CTA: up)
        const bool gate_up = q.epi_mode == 1;
        const int n0 = gate_up ? it.nt * 128 : it.nt * 256 + (int)rank * 128;
        const int pa_mn = q.a_mn, pb_mn = q.b_mn;
        const int nmain = it.kb1 - it.kb0;
        const int nkb = nmain + it.next;
        KCursor cur(q, it.kb0, nmain);
        for (int i = 0; i < nkb; ++i) {
          const CUtensorMap *ma, *mb;
          int kel;
          cur.take(ma, mb, kel);
          if (!mbar_wait_fast(empty_bar(stage), phase ^ 1u, abort_flag, g.status, 400)) { ok = false; break; }
          const uint32_t fb = full0 + 8u * stage;   // the even CTA's barrier
          // one announcement covers the bytes of both operands of both CTAs (bytes may land before it)
          if (rank == 0 && do_a) mbar_arrive_expect_tx(full_bar(stage), 2u * (uint32_t)kStage);
          const uint32_t sA = smem0 + stage * kStage, sB = sA + kStageA;
          if (do_a) {
            if (!pa_mn) {
              tma_load_2d_pair(sA, ma, fb, kel, m0);
            } else {
#pragma unroll
              for (int b = 0; b < 2; ++b) tma_load_2d_pair(sA + b * 8192, ma, fb, m0 + b * 64, kel);
            }
          } else {
            if (!pb_mn) {
              int nrow = n0;
              if (gate_up) {
                // main blocks: each CTA its own frozen weight; the rank-r blocks of a projection meet zeros in
                // the other projection's half (rows beyond the tensor are filled with zeros by the copy)
                if (cur.seg == 0) { if (rank) mb = &q.tmXb[1]; }
                else if ((cur.seg == 1) == (rank == 1)) nrow = kRowsBeyond;
              }
              tma_load_2d_pair(sB, mb, fb, kel, nrow);
            } else {
#pragma unroll
              for (int b = 0; b < 2; ++b) tma_load_2d_pair(sB + b * 8192, mb, fb, n0 + b * 64, kel);
            }
          }
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (dealer) { item = next_item; next_item = drawn; }
      }
      if (!ok && rank == 0) {
        long long n = issued < kStages ? issued : kStages;
        for (long long k = 0; k < n; ++k) {
          long long idx = issued - 1 - k;
          int s = (int)(idx % kStages);
          uint32_t ph = (uint32_t)((idx / kStages) & 1);
          const unsigned long long t0 = globaltimer_ns();
          while (!mbar_try(full_bar(s), ph) && globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (even CTA only) =====================
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int local = 0, sslot = 0;
      uint32_t sphase = 0;
      bool ok = true;
      for (; ok; ++local) {
        int item;
        if (!ring_take(sslot, sphase, 510, item)) { ok = false; break; }
        ring_release(sslot, sphase);
        if (item >= g.n_items) break;
        const Item it = decode_item_pair(g, item);
        const DevProb &q = g.p[it.p];
        const int nkb = (it.kb1 - it.kb0) + it.next;
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, g.status, 500)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * 256);
        const int a_mn = q.a_mn, b_mn = q.b_mn;
        const uint32_t idesc = instr_desc_pair(a_mn, b_mn);
        const uint64_t a_tmpl = smem_desc_template(a_mn), b_tmpl = smem_desc_template(b_mn);
        const uint32_t a_step = smem_desc_kstep(a_mn), b_step = smem_desc_kstep(b_mn);
        for (int i = 0; i < nkb; ++i) {
          if (!mbar_wait_fast(full_bar(stage), phase, abort_flag, g.status, 501)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_lo = (smem0 + stage * kStage) >> 4, b_lo = a_lo + (kStageA >> 4);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            tc_mma_bf16_pair(d_tmem, a_tmpl | (uint64_t)(a_lo + kk * a_step), b_tmpl | (uint64_t)(b_lo + kk * b_step),
                             idesc, (i | kk) != 0 ? 1u : 0u);
          tc_commit_pair(empty_bar(stage));   // frees this stage in both CTAs
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit_pair(tfull_bar(acc));  // accumulator complete, both CTAs
      }
      if (!ok) {
        tc_commit_pair(drain_bar);
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try(drain_bar, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else {
    // ===================== epilogue (warps 2..5, both CTAs) =====================
    const int quarter = warp & 3;
    int local = 0, sslot = 0;
    uint32_t sphase = 0;
    bool ok = true;
    const uint32_t my_stage = out_stage0 + (uint32_t)quarter * (2u * kOutBox);
    uint32_t chunk_no = 0;   // chunks this warp has staged so far (selects the buffer)
    for (; ok; ++local) {
      int item;
      ok = __all_sync(0xffffffffu, ring_take(sslot, sphase, 610, item));
      if (!ok) break;
      __syncwarp();
      if (lane == 0) ring_release(sslot, sphase); else if (++sslot == kSched) { sslot = 0; sphase ^= 1u; }
      __syncwarp();
      if (item >= g.n_items) break;
      const Item it = decode_item_pair(g, item);
      const DevProb &q = g.p[it.p];
      const int n0 = q.epi_mode == 1 ? it.nt * 128 : it.nt * 256;
      const int acc = local & 1;
      const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, g.status, 600)) { ok = false; break; }
      tc_fence_after();
      const int row0 = it.m0 + (int)rank * 128 + quarter * 32;   // first of this warp's 32 rows
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 256);
      uint32_t v[32], w[32];
      if (q.epi_mode != 0) {
        // Gating fused into the epilogue.  32 columns at a time: the accumulator values (and, backwards, the saved
        // gate and up values of the same elements) are combined in registers, every output gets a 32 x 32 bf16 box
        // (64-byte rows, not swizzled) in this warp's staging area, and bulk tensor stores write the boxes out.
        const bool fwd = q.epi_mode == 1;
        const int row = row0 + lane;
#pragma unroll 1
        for (int c0 = 0; c0 < (fwd ? 128 : 256); c0 += 32) {
          const int col = n0 + c0;
          tmem_ld32(t_row + c0, v);                              // forward: gate; backward: dh
          if (fwd) tmem_ld32(t_row + 128 + c0, w);               // forward: up
          uint4 gq[4], uq[4];
          if (!fwd) {                                            // backward: saved gate and up, 64 bytes each
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              gq[j] = make_uint4(0u, 0u, 0u, 0u); uq[j] = gq[j];
              if (row < q.M && col + 8 * j + 8 <= q.N) {
                const long long off = (long long)row * q.out_s0 + col + 8 * j;
                gq[j] = *reinterpret_cast<const uint4 *>(q.epi_in0 + off);
                uq[j] = *reinterpret_cast<const uint4 *>(q.epi_in1 + off);
              }
            }
          }
          if (lane == 0) bulk_wait_group_read<0>();              // the previous boxes have been read out
          tmem_ld_wait();
          __syncwarp();
          const uint32_t box0 = my_stage + (uint32_t)lane * 64u, box1 = box0 + 2048u, box2 = box0 + 4096u;
          if (fwd) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint32_t hh[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float gv = __uint_as_float(v[8 * j + e]), uv = __uint_as_float(w[8 * j + e]);
                hh[e] = __float_as_uint(gv * __fdividef(1.f, 1.f + __expf(-gv)) * uv);
              }
              st_shared_v4(box0 + 16u * j, pack_bf16x2(v[8 * j], v[8 * j + 1]), pack_bf16x2(v[8 * j + 2], v[8 * j + 3]),
                           pack_bf16x2(v[8 * j + 4], v[8 * j + 5]), pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
              st_shared_v4(box1 + 16u * j, pack_bf16x2(w[8 * j], w[8 * j + 1]), pack_bf16x2(w[8 * j + 2], w[8 * j + 3]),
                           pack_bf16x2(w[8 * j + 4], w[8 * j + 5]), pack_bf16x2(w[8 * j + 6], w[8 * j + 7]));
              st_shared_v4(box2 + 16u * j, pack_bf16x2(hh[0], hh[1]), pack_bf16x2(hh[2], hh[3]), pack_bf16x2(hh[4], hh[5]),
                           pack_bf16x2(hh[6], hh[7]));
            }
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const __nv_bfloat162 *g2 = reinterpret_cast<const __nv_bfloat162 *>(&gq[j]);
              const __nv_bfloat162 *u2 = reinterpret_cast<const __nv_bfloat162 *>(&uq[j]);
              uint32_t dg[8], du[8];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 gf = __bfloat1622float2(g2[e]), uf = __bfloat1622float2(u2[e]);
                const float d0 = __uint_as_float(v[8 * j + 2 * e]), d1 = __uint_as_float(v[8 * j + 2 * e + 1]);
                const float s0 = __fdividef(1.f, 1.f + __expf(-gf.x)), s1 = __fdividef(1.f, 1.f + __expf(-gf.y));
                dg[2 * e] = __float_as_uint(d0 * uf.x * s0 * (1.f + gf.x * (1.f - s0)));
                dg[2 * e + 1] = __float_as_uint(d1 * uf.y * s1 * (1.f + gf.y * (1.f - s1)));
                du[2 * e] = __float_as_uint(d0 * gf.x * s0);
                du[2 * e + 1] = __float_as_uint(d1 * gf.y * s1);
              }
              st_shared_v4(box0 + 16u * j, pack_bf16x2(dg[0], dg[1]), pack_bf16x2(dg[2], dg[3]), pack_bf16x2(dg[4], dg[5]),
                           pack_bf16x2(dg[6], dg[7]));
              st_shared_v4(box1 + 16u * j, pack_bf16x2(du[0], du[1]), pack_bf16x2(du[2], du[3]), pack_bf16x2(du[4], du[5]),
                           pack_bf16x2(du[6], du[7]));
            }
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0 && row0 < q.M && col < q.N) {
            tma_store_2d(&q.tmOut, my_stage, col, row0);
            tma_store_2d(&q.tmXa[1], my_stage + 2048u, col, row0);
            if (fwd) tma_store_2d(&q.tmXa[2], my_stage + 4096u, col, row0);
            bulk_commit_group();
          }
        }
        if (lane == 0) bulk_wait_group_read<0>();   // the plain path below alternates buffers on its own count
        __syncwarp();
      } else
#pragma unroll 1
      for (int c0 = 0; c0 < 256; c0 += 64, ++chunk_no) {
        tmem_ld32(t_row + c0, v);
        tmem_ld32(t_row + c0 + 32, w);
        // the store that read this buffer two chunks ago must be done with it
        if (lane == 0) bulk_wait_group_read<1>();
        tmem_ld_wait();
        __syncwarp();
        const uint32_t buf = my_stage + (chunk_no & 1u) * (uint32_t)kOutBox;
        const uint32_t rowp = buf + (uint32_t)lane * 128u;
        const uint32_t sw = (uint32_t)(lane & 7);
#pragma unroll
        for (int j = 0; j < 4; ++j) {   // 16-byte piece j of the row holds columns 8j .. 8j+7, stored at piece j ^ (row % 8)
          st_shared_v4(rowp + (((uint32_t)j ^ sw) << 4), pack_bf16x2(v[8 * j], v[8 * j + 1]),
                       pack_bf16x2(v[8 * j + 2], v[8 * j + 3]), pack_bf16x2(v[8 * j + 4], v[8 * j + 5]),
                       pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
          st_shared_v4(rowp + (((uint32_t)(j + 4) ^ sw) << 4), pack_bf16x2(w[8 * j], w[8 * j + 1]),
                       pack_bf16x2(w[8 * j + 2], w[8 * j + 3]), pack_bf16x2(w[8 * j + 4], w[8 * j + 5]),
                       pack_bf16x2(w[8 * j + 6], w[8 * j + 7]));
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < q.M && n0 + c0 < q.N) {   // rows and columns beyond the tensor are clipped by the store
          tma_store_2d(&q.tmOut, buf, n0 + c0, row0);
          bulk_commit_group();
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(acc), 0));
    }
    if (lane == 0) bulk_wait_group_all();   // every store of this warp has left shared memory and is complete
    __syncwarp();
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // neither CTA leaves while the other may still signal its barriers
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                 : "memory");
  }
  // the last pair to finish re-arms the item counter for the next launch on this workspace
  if (rank == 0 && threadIdx.x == 0) {
    __threadfence();
    const int done = atomicAdd(&g.status->sched_done, 1);
    if (done == n_pairs - 1) {
      g.status->sched_next = 0;
      g.status->sched_done = 0;
      __threadfence();
    }
  }
}

}  // namespace pair

// ------------------------------------------------------------------ decode in one kernel (cluster split-K)
// The decode-time forward of up to kDclMaxProj projections in a single launch.  A cluster of S CTAs
// owns one 128-row tile of one projection's output at a time; CTA r of the cluster streams the r-th
// part of the tile's k-blocks of W0 (TMA, evict-first) against x and accumulates its partial tile in
// TMEM.  The partials never leave the chip: CTAs 1 .. S-1 send theirs from registers into CTA 0's
// shared memory (st.async, counted by an mbarrier of CTA 0), CTA 0 adds them to its own in rank order
// (deterministic) and writes y.  The rank-r term rides in the same accumulators as extension k-blocks
// (B tile x (s u)^T) at the end of the tile's k-block sequence.  u = A x^T is itself one more item per
// projection (the rows of A as the streamed operand): its cluster writes s*u as bf16 to scratch and
// raises a flag (zero again when the launch ends) that the other clusters' producers check before they
// load extension operands.  The u items are dealt first, so each is the first item of its cluster
// and waits for nothing.  Items are handed out dynamically: CTA 0's producer draws them from a global
// counter and writes them into every CTA's item ring.
namespace dcl {

#ifndef TL_DCL_EARLY
#define TL_DCL_EARLY 1
#endif

constexpr int kSub = kStageA + 16 * BK * 2;        // one k-block: 128 x 64 of W0 + 16 x 64 of x
// Shared memory of a CTA: the operand ring (n_stages stages of KPS k-blocks), then room for the partial
// tiles of the S - 1 other CTAs (used in CTA 0 only, but every CTA of a launch has the same layout;
// 16 bytes per row and four tokens), then barriers and the item ring.  The host picks KPS and n_stages
// so that the ring is as deep as the 227 KB allow: bytes in flight are what keeps HBM busy.
constexpr int kMaxStages = 6;
constexpr int kSmemLimit = 227 * 1024;
__host__ __device__ constexpr int recv_bytes(int S, int n_tokens) { return (S - 1) * 128 * 16 * ((n_tokens + 3) / 4); }
inline int stages_that_fit(int S, int kps, int n_tokens) {
  const int n = (kSmemLimit - 2048 - recv_bytes(S, n_tokens)) / (kps * kSub);
  return n > kMaxStages ? kMaxStages : n;
}
constexpr int kTmemCols = 32;
constexpr int kDclMaxProj = 8;
constexpr int kRing = 8;    // items the dealer may run ahead of the slowest reader in the cluster

// The launch's problems travel as a DevGroup: role (DevProb::pad) 0 = a projection's y (A-op W0, B-op x,
// extension A-op B, B-op s*u; out = y [n, d_out] bf16), 1 = its u (A-op A, B-op x; out = s*u [n, r] bf16,
// scale in epi_scale); DevProb::pad3 = the projection's slot among the ready flags.
struct DclParams {
  int n_tokens, n_stages;
};

template <int S, int KPS>
__global__ void __launch_bounds__(kThreads, 1)
    decode_cluster_kernel(const __grid_constant__ DevGroup g, const DclParams prm) {
  constexpr int kKps = KPS, kStage = kKps * kSub;
  const int kStages = prm.n_stages;   // runtime: what fits beside the receive buffer
  const int nv = (prm.n_tokens + 3) >> 2;   // 16-byte pieces of a row that carry tokens
  const int slot_bytes = 128 * 16 * nv;     // one peer's partial tile in the receive buffer
  const int kRecvBytes = (S - 1) * slot_bytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_al = smem_raw + (smem0 - smem_u32(smem_raw));
  const uint32_t recv0 = smem0 + kStages * kStage;               // CTA 0: partial tiles of CTAs 1 .. S-1
  const float *recv_ptr = reinterpret_cast<const float *>(smem_al + kStages * kStage);
  const uint32_t bar0 = recv0 + kRecvBytes;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + 2 + a); };
  const uint32_t part_full = bar0 + 8u * (2 * kMaxStages + 4);      // used in CTA 0: the peers' partials have landed
  const uint32_t part_free = bar0 + 8u * (2 * kMaxStages + 5);      // one per peer: CTA 0 has read its last partial
  const uint32_t drain_bar = bar0 + 8u * (2 * kMaxStages + 6);
  auto sfull_bar = [&](int s) { return bar0 + 8u * (2 * kMaxStages + 7 + s); };            // one per CTA
  auto sempty_bar = [&](int s) { return bar0 + 8u * (2 * kMaxStages + 7 + kRing + s); };  // used in CTA 0
  uint8_t *misc = smem_al + kStages * kStage + kRecvBytes + 512;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(misc);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(misc + 4);
  volatile int *sched_ring = reinterpret_cast<volatile int *>(misc + 16);
  const uint32_t ring0 = bar0 + 512 + 16;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int cluster_id = blockIdx.x / S, n_clusters = gridDim.x / S;
  int *flags = &g.status->pad[0];
  // every role but CTA 0's producer takes its items from the ring: 6 per CTA
  constexpr int kRingReaders = 6 * S - 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    mbar_init(part_full, 4);       // one lane of each epilogue warp of CTA 0 (each also announces its share of the bytes)
    mbar_init(part_free, 4);       // one lane of each epilogue warp of CTA 0
    mbar_init(drain_bar, 1);
    for (int s = 0; s < kRing; ++s) { mbar_init(sfull_bar(s), 1); mbar_init(sempty_bar(s), kRingReaders); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                 "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the peers' barriers are initialised before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Ordering against the kernels ahead on the stream.  Everything this kernel reads may have been written by them
  // EXCEPT the frozen weights W0, which nothing ever writes: the producer thread requests the W0 tiles of its
  // cluster's first item before it waits for the predecessors (the requests then overlap the predecessor's last
  // items and the completion hand-over between the two grids), every other thread waits here.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!(TL_DCL_EARLY && warp == 0)) asm volatile("griddepcontrol.wait;" ::: "memory");

  // this CTA's share of an item.  The streamed operand's k-blocks are dealt to the S CTAs in chunks of KPS
  // (one pipeline stage) round-robin, so at any time the cluster reads neighbouring pieces of the same
  // rows of W0 (the same DRAM pages): CTA r takes chunks r, r + S, ...  nmain = its streamed k-blocks.
  // The extension blocks go to the last CTA, which never has more streamed blocks than the others.
  auto share_of = [&](int item, int &p, int &m0, int &nmain, int &next) {
    p = 0;
    while (p + 1 < g.n_prob && item >= g.p[p + 1].item_start) ++p;
    const DevProb &q = g.p[p];
    m0 = (item - q.item_start) * BM;
    const int chunks = (q.kb_main + kKps - 1) / kKps;
    const int mine = rank < chunks ? (chunks - rank + S - 1) / S : 0;
    nmain = mine * kKps;
    if (mine > 0 && (chunks - 1) % S == rank) nmain -= chunks * kKps - q.kb_main;   // the ragged last chunk
    next = (rank == S - 1) ? q.kb_ext : 0;
  };
  // take the next item from this CTA's ring (written by CTA 0's producer) and hand the slot back
  auto ring_take = [&](int &sslot, uint32_t &sphase, int where, int &item) -> bool {
    if (!mbar_wait_acq_cluster(sfull_bar(sslot), sphase, abort_flag, g.status, where)) return false;
    item = sched_ring[sslot];
    return true;
  };
  auto ring_release = [&](int &sslot, uint32_t &sphase) {
    mbar_arrive_remote_plain(mapa_shared(sempty_bar(sslot), 0));
    if (++sslot == kRing) { sslot = 0; sphase ^= 1u; }
  };

  if (warp == 0) {
    // ===================== TMA producer; in CTA 0 it also deals the items =====================
    if (lane == 0) {
      int stage = 0, sslot = 0;
      uint32_t phase = 0, sphase = 0;
      long long issued = 0;
      bool ok = true;
      int item = cluster_id;
      const uint64_t stream_policy = l2_policy_evict_first();
      uint32_t ready_mask = 0;   // projections whose s*u this thread has seen complete
      // CTA 0: write an item into every CTA's ring (the slot must have been handed back by all its readers)
      auto deal = [&](int it) -> bool {
        if (!mbar_wait(sempty_bar(sslot), sphase ^ 1u, abort_flag, g.status, 830)) return false;
#pragma unroll
        for (int r = 0; r < S; ++r) st_cluster_s32(mapa_shared(ring0 + 4u * sslot, (uint32_t)r), it);
#pragma unroll
        for (int r = 0; r < S; ++r)   // release at cluster scope: the store above is visible to whoever sees this arrival
          mbar_arrive_cluster(mapa_shared(sfull_bar(sslot), (uint32_t)r));
        if (++sslot == kRing) { sslot = 0; sphase ^= 1u; }
        return true;
      };
      // The cluster's first item is known without the counter (cluster c starts on item c).  When it is a y item,
      // the W0 part of its first stages is requested now, the x part right after the wait below.
      int pre_chunks = 0;
      if (TL_DCL_EARLY) {
        if (item < g.n_items) {
          int p, m0, nmain, next;
          share_of(item, p, m0, nmain, next);
          const DevProb &q = g.p[p];
          if (q.pad == 0) {   // role 0: the streamed operand is W0
            pre_chunks = nmain / kKps;   // whole stages made of streamed k-blocks only
            if (pre_chunks > kStages) pre_chunks = kStages;
            for (int c = 0; c < pre_chunks; ++c) {
              mbar_arrive_expect_tx(full_bar(c), (uint32_t)(kKps * kSub));
              for (int j = 0; j < kKps; ++j) {
                const int kel = ((c * S + rank) * kKps + j) * BK;
                tma_load_2d_hint(smem0 + c * kStage + j * kSub, &q.tmA, full_bar(c), kel, m0, stream_policy);
              }
            }
          }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (pre_chunks) {
          int p, m0, nmain, next;
          share_of(item, p, m0, nmain, next);
          const DevProb &q = g.p[p];
          for (int c = 0; c < pre_chunks; ++c)
            for (int j = 0; j < kKps; ++j) {
              const int kel = ((c * S + rank) * kKps + j) * BK;
              tma_load_2d(smem0 + c * kStage + j * kSub + kStageA, &q.tmB, full_bar(c), kel, 0);
            }
        }
      }
      // CTA 0 deals one item ahead (the peers learn the next item before this CTA starts loading the
      // current one) and draws two ahead, so the counter's round trip is never waited for
      int next_item = 0, drawn = 0;
      if (rank == 0) {
        next_item = n_clusters + atomicAdd(&g.status->sched_next, 1);
        ok = deal(item);
      }
      while (ok) {
        if (rank == 0) {
          if (item >= g.n_items) break;   // the end marker has been passed on
          if (!deal(next_item)) { ok = false; break; }
          drawn = next_item < g.n_items ? n_clusters + atomicAdd(&g.status->sched_next, 1) : next_item;
        } else {
          if (!ring_take(sslot, sphase, 831, item)) { ok = false; break; }
          ring_release(sslot, sphase);
          if (item >= g.n_items) break;
        }
        int p, m0, nmain, next;
        share_of(item, p, m0, nmain, next);
        const DevProb &q = g.p[p];
        const int nkb = nmain + next;
        bool u_ready = (next == 0) || ((ready_mask >> q.pad3) & 1u);
        // the ready flags are requested now and looked at when the extension blocks come up
        int4 f0 = make_int4(0, 0, 0, 0), f1 = f0;
        if (!u_ready) { f0 = ld_volatile_i4(flags); f1 = ld_volatile_i4(flags + 4); }
        for (int i0 = 0; ok && i0 < nkb; i0 += kKps) {
          const int cnt = (nkb - i0 < kKps) ? nkb - i0 : kKps;
          if (pre_chunks > 0) {   // this stage of the first item was requested before the loop
            --pre_chunks;
            ++issued;
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
            continue;
          }
          if (!u_ready && i0 + cnt > nmain) {
            // s*u of this projection must be complete (another cluster writes it): bounded wait on its flag.
            // One pass reads the flags of all projections, so each is usually waited for once per CTA.
            const unsigned long long t0 = globaltimer_ns();
            while (true) {
              const int f[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
#pragma unroll
              for (int w = 0; w < 8; ++w) ready_mask |= (f[w] != 0 ? 1u : 0u) << w;
              if ((ready_mask >> q.pad3) & 1u) break;
              f0 = ld_volatile_i4(flags); f1 = ld_volatile_i4(flags + 4);
              if (*abort_flag || globaltimer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                if (atomicCAS(&g.status->code, 0, (int)TEMPLORA_ERR_TIMEOUT) == 0) g.status->where = 801;
                __threadfence();
                ok = false;
                break;
              }
            }
            if (!ok) break;
            __threadfence();       // acquire side of the flag
            fence_async_proxy();   // those generic-proxy writes are read by the TMA loads below
            u_ready = true;
          }
          if (!mbar_wait_fast(empty_bar(stage), phase ^ 1u, abort_flag, g.status, 800)) { ok = false; break; }
          mbar_arrive_expect_tx(full_bar(stage), (uint32_t)(cnt * kSub));
          for (int j = 0; j < cnt; ++j) {
            const int i = i0 + j;
            const uint32_t sA = smem0 + stage * kStage + j * kSub, sB = sA + kStageA;
            if (i < nmain) {
              const int kel = (((i / kKps) * S + rank) * kKps + i % kKps) * BK;
              tma_load_2d_hint(sA, &q.tmA, full_bar(stage), kel, m0, stream_policy);   // read exactly once
              tma_load_2d(sB, &q.tmB, full_bar(stage), kel, 0);
            } else {
              const int kel = (i - nmain) * BK;
              tma_load_2d(sA, &q.tmAe, full_bar(stage), kel, m0);
              tma_load_2d(sB, &q.tmBe, full_bar(stage), kel, 0);
            }
          }
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (rank == 0) { item = next_item; next_item = drawn; }
      }
      if (!ok) {
        // wait (bounded) for the copies this thread still has in flight before the CTA may exit
        long long n = issued < kStages ? issued : kStages;
        for (long long k = 0; k < n; ++k) {
          const long long idx = issued - 1 - k;
          const unsigned long long t0 = globaltimer_ns();
          while (!mbar_try(full_bar((int)(idx % kStages)), (uint32_t)((idx / kStages) & 1)) &&
                 globaltimer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      int stage = 0, local = 0, sslot = 0;
      uint32_t phase = 0, sphase = 0;
      bool ok = true;
      const uint32_t idesc = instr_desc(16, 0, 0);
      const uint64_t tmpl = smem_desc_template(0);
      const uint32_t kstep = smem_desc_kstep(0);
      while (ok) {
        int item;
        if (!ring_take(sslot, sphase, 812, item)) { ok = false; break; }
        ring_release(sslot, sphase);
        if (item >= g.n_items) break;
        int p, m0, nmain, next;
        share_of(item, p, m0, nmain, next);
        const int nkb = nmain + next;
        if (nkb == 0) continue;   // nothing of this item falls to this CTA: its epilogue parks zeros
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        ++local;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, g.status, 810)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * 16);
        for (int i0 = 0; i0 < nkb; i0 += kKps) {
          const int cnt = (nkb - i0 < kKps) ? nkb - i0 : kKps;
          if (!mbar_wait_fast(full_bar(stage), phase, abort_flag, g.status, 811)) { ok = false; break; }
          tc_fence_after();
          for (int j = 0; j < cnt; ++j) {
            const uint32_t a_lo = (smem0 + stage * kStage + j * kSub) >> 4, b_lo = a_lo + (kStageA >> 4);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              tc_mma_bf16(d_tmem, tmpl | (uint64_t)(a_lo + kk * kstep), tmpl | (uint64_t)(b_lo + kk * kstep), idesc,
                          (i0 | j | kk) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(tfull_bar(acc));
      }
      if (!ok) {
        tc_commit(drain_bar);   // let MMAs already issued finish before TMEM is released
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try(drain_bar, 0) && globaltimer_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else {
    // ===================== epilogue and in-cluster reduction (warps 2..5) =====================
    const int quarter = warp & 3;   // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    const int row_in_tile = quarter * 32 + lane;
    int local = 0, sslot = 0;
    uint32_t sphase = 0;
    bool ok = true;
    for (int seq = 0; ok; ++seq) {   // seq: items this cluster has taken (phase of the part_* barriers)
      int item;
      ok = __all_sync(0xffffffffu, ring_take(sslot, sphase, 823, item));
      if (!ok) break;
      __syncwarp();
      if (lane == 0) ring_release(sslot, sphase); else if (++sslot == kRing) { sslot = 0; sphase ^= 1u; }
      __syncwarp();
      if (item >= g.n_items) break;
      int p, m0, nmain, next;
      share_of(item, p, m0, nmain, next);
      const DevProb &q = g.p[p];
      uint32_t v[32];
#pragma unroll
      for (int c = 0; c < 16; ++c) v[c] = 0u;
      if (nmain + next > 0) {
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        ++local;
        ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag, g.status, 820));
        if (!ok) break;
        tc_fence_after();
        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 16), v);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
        __syncwarp();
      }
      if (rank != 0) {
        // send this row's partial sums into CTA 0's shared memory, once CTA 0 has read the previous ones
        ok = __all_sync(0xffffffffu, mbar_wait(part_free, (uint32_t)(seq & 1) ^ 1u, abort_flag, g.status, 821));
        if (!ok) break;
        const uint32_t dst = mapa_shared(recv0 + (uint32_t)((rank - 1) * slot_bytes + row_in_tile * 16 * nv), 0);
        const uint32_t bar = mapa_shared(part_full, 0);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (c < nv) st_async_v4(dst + 16u * c, v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3], bar);
        continue;
      }

      // CTA 0: wait for the S - 1 other partials and add them in rank order (deterministic)
      if (lane == 0) mbar_arrive_expect_tx(part_full, (uint32_t)((S - 1) * 32 * 16 * nv));
      __syncwarp();   // lane 0 must have arrived before the warp starts polling: the barrier needs that arrival
      ok = __all_sync(0xffffffffu, mbar_wait(part_full, (uint32_t)(seq & 1), abort_flag, g.status, 822));
      if (!ok) break;
      float sum[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) sum[c] = __uint_as_float(v[c]);
#pragma unroll
      for (int r = 1; r < S; ++r) {
        const float4 *src = reinterpret_cast<const float4 *>(recv_ptr + (r - 1) * (slot_bytes / 4) + row_in_tile * 4 * nv);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (c < nv) {
            const float4 t = src[c];
            sum[4 * c] += t.x; sum[4 * c + 1] += t.y; sum[4 * c + 2] += t.z; sum[4 * c + 3] += t.w;
          }
      }
      __syncwarp();
      if (lane == 0) {
#pragma unroll
        for (int r = 1; r < S; ++r) mbar_arrive_remote_plain(mapa_shared(part_free, (uint32_t)r));
      }
      __syncwarp();
      const int row = m0 + row_in_tile;
      const bool is_u = q.pad == 1;
      if (row < q.M) {
        __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(q.out) + row;
        const float sc = is_u ? q.epi_scale : 1.f;
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (i < prm.n_tokens) out[(long long)i * q.out_s1] = __float2bfloat16_rn(sc * sum[i]);
      }
      if (is_u) {   // publish s*u: the last of the four warps to finish its rows raises the flag
        __threadfence();
        fence_async_proxy();
        __syncwarp();
        if (lane == 0) {
          int *arrived = flags + kDclMaxProj + q.pad3;
          if (atomicAdd(arrived, 1) == 3) {
            *arrived = 0;
            __threadfence();
            st_release_gpu(flags + q.pad3, 1);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // no CTA leaves while a peer may still read its partial or signal its barriers
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
  }
  // the last cluster to finish re-arms the item counter and the ready flags for the next launch on this
  // workspace (nothing of the launch depends on a number the host hands in, so a recorded launch can be replayed)
  if (rank == 0 && threadIdx.x == 0) {
    __threadfence();
    const int done = atomicAdd(&g.status->sched_done, 1);
    if (done == n_clusters - 1) {
      for (int w = 0; w < kDclMaxProj; ++w) flags[w] = 0;
      g.status->sched_next = 0;
      g.status->sched_done = 0;
      __threadfence();
    }
  }
}

}  // namespace dcl


}  // namespace

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
    if (qres != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// 2-D bf16 tensor [outer][inner] with row pitch `pitch` elements; box = 64 x box_outer, 128B swizzle.
// Encoded descriptors are kept in a per-thread table: a descriptor depends only on (address, extents,
// pitch, box), weights and state buffers keep their addresses from call to call, and encoding is a
// sizeable part of the host time of a small call (a decode step of one projection is ~5 us of GPU work).
struct MapKey {
  const void *ptr;
  long long inner, outer, pitch;
  int box_outer, box_inner;   // box_inner 64: 128-byte swizzle (operand tiles, plain outputs); 32: not swizzled
  bool operator==(const MapKey &o) const {
    return ptr == o.ptr && inner == o.inner && outer == o.outer && pitch == o.pitch && box_outer == o.box_outer &&
           box_inner == o.box_inner;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey &k) const {
    size_t h = reinterpret_cast<size_t>(k.ptr) * 0x9E3779B97F4A7C15ull;
    h ^= (size_t)k.inner * 0xC2B2AE3D27D4EB4Full + (size_t)k.outer * 0x165667B19E3779F9ull + (size_t)k.pitch * 31 +
         (size_t)k.box_outer + 1024u * (size_t)k.box_inner;
    return h ^ (h >> 29);
  }
};
bool make_map(CUtensorMap *m, const void *ptr, long long inner, long long outer, long long pitch, int box_outer,
              int box_inner) {
  static thread_local std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  const MapKey key{ptr, inner, outer, pitch, box_outer, box_inner};
  auto it = cache.find(key);
  if (it != cache.end()) {
    *m = it->second;
    return true;
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t gstr[1] = {(cuuint64_t)pitch * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, box_inner == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() >= 8192) cache.clear();
  cache.emplace(key, *m);
  return true;
}

// operand [rows = M or N][K] (mn = 0) or [K][M or N] (mn = 1)
bool make_operand_map(CUtensorMap *m, const void *ptr, long long mn_extent, long long k_extent, long long ld, int mn,
                      int tile_mn) {
  if (!mn) return make_map(m, ptr, k_extent, mn_extent, ld, tile_mn);
  return make_map(m, ptr, mn_extent, k_extent, ld, 64);
}

// Per-stream cap on the SMs the persistent kernels occupy (parallelized deployment: the chunk update
// and the decode stream share the GPU).  0 / absent = no cap.
std::mutex g_limit_mu;
std::unordered_map<cudaStream_t, int> g_stream_limit;
int stream_sm_limit(cudaStream_t st, int sm_count) {
  std::lock_guard<std::mutex> lk(g_limit_mu);
  auto it = g_stream_limit.find(st);
  if (it == g_stream_limit.end() || it->second <= 0 || it->second > sm_count) return sm_count;
  return it->second;
}

DeviceInfo *device_info() {
  static DeviceInfo info[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  DeviceInfo &d = info[dev];
  if (d.sm_count == 0) {
    int sm = 0, major = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return nullptr;
    d.cc_major = major;
    d.sm_count = sm;
  }
  return &d;
}

namespace {

template <int BN>
templora_status_t launch(const DevGroup &g, DeviceInfo *di, int slot, cudaStream_t st) {
  if (!di->attr_set[slot]) {
    TL_CUDA_CHECK(cudaFuncSetAttribute(tc_gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN>::kSmemBytes));
    di->attr_set[slot] = true;
  }
  const int sms = stream_sm_limit(st, di->sm_count);
  int grid = g.n_items < sms ? g.n_items : sms;
  {
    LaunchScope scope(g.p[0].epi_mask ? kKindTcDropoutTerm
                                       : (BN == 256 ? kKindTcMain : (BN == 64 ? kKindTcSkinny : kKindTcDecode)), st);
    TL_CUDA_CHECK(launch_pdl(tc_gemm_kernel<BN>, dim3(grid), dim3(kThreads2), Cfg<BN>::kSmemBytes, st, g));
  }
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

templora_status_t launch_pair(const DevGroup &g, DeviceInfo *di, cudaStream_t st) {
  if (!di->pair_attr_set) {
    TL_CUDA_CHECK(cudaFuncSetAttribute(pair::tc_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       pair::kSmemBytes));
    di->pair_attr_set = true;
  }
  int pairs = stream_sm_limit(st, di->sm_count) / 2;
  if (pairs < 1) pairs = 1;
  if (g.n_items < pairs) pairs = g.n_items;
  {
    LaunchScope scope(kKindTcMain, st);
    TL_CUDA_CHECK(launch_pdl(pair::tc_gemm_pair_kernel, dim3(2 * pairs), dim3(pair::kPairThreads), pair::kSmemBytes, st, g));
  }
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

// ---- decode in one kernel: launch ------------------------------------------------
// Clusters of S CTAs of this kernel variant that fit on the device at once (asked once per device).
template <int S, int KPS>
int decode_cluster_fit(DeviceInfo *di, int slot) {
  if (di->dcl_clusters[slot] != 0) return di->dcl_clusters[slot];
  auto kernel = dcl::decode_cluster_kernel<S, KPS>;
  di->dcl_clusters[slot] = -1;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dcl::kSmemLimit) != cudaSuccess) return -1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.gridDim = dim3(di->sm_count / S * S);
  cfg.dynamicSmemBytes = dcl::kSmemLimit;   // one CTA per SM whatever the exact size
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int fit = 0;
  if (cudaOccupancyMaxActiveClusters(&fit, kernel, &cfg) != cudaSuccess || fit < 1) return -1;
  di->dcl_clusters[slot] = fit;
  return fit;
}

template <int S, int KPS>
templora_status_t launch_decode_cluster(const DevGroup &g, dcl::DclParams prm, DeviceInfo *di, int slot, cudaStream_t st,
                                        int min_clusters) {
  auto kernel = dcl::decode_cluster_kernel<S, KPS>;
  prm.n_stages = dcl::stages_that_fit(S, KPS, prm.n_tokens);
  if (prm.n_stages < 2) return TEMPLORA_ERR_UNSUPPORTED;
  int clusters = decode_cluster_fit<S, KPS>(di, slot);
  const int cap = stream_sm_limit(st, di->sm_count) / S;
  if (clusters > cap) clusters = cap;
  if (clusters > g.n_items) clusters = g.n_items;
  if (clusters < 1 || clusters < min_clusters) return TEMPLORA_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(clusters * S);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = prm.n_stages * KPS * dcl::kSub + dcl::recv_bytes(S, prm.n_tokens) + 2048;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  {
    LaunchScope scope(kKindTcDecode, st);
    TL_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kernel, g, prm));
  }
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

}  // namespace

// ------------------------------------------------------------------ bounded-wait self-test
// One CTA waits, with the same poll / timer / status-record steps as the GEMM kernels' waits, on an
// mbarrier that nothing will ever arrive at.  After limit_ns it must record TEMPLORA_ERR_TIMEOUT and
// return, leaving the context usable.
namespace {
__global__ void wait_selftest_kernel(DeviceStatus *st, unsigned long long limit_ns, int where) {
  __shared__ __align__(8) unsigned long long bar_storage;
  const uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const unsigned long long t0 = globaltimer_ns();
    bool done = false;
    while (!done) {
      for (int i = 0; i < 256 && !done; ++i) done = mbar_try(bar, 0);
      if (!done && globaltimer_ns() - t0 > limit_ns) {
        if (atomicCAS(&st->code, 0, (int)TEMPLORA_ERR_TIMEOUT) == 0) st->where = where;
        __threadfence();
        break;
      }
    }
  }
}
}  // namespace

templora_status_t tc_wait_selftest(DeviceStatus *status, unsigned long long limit_ns, cudaStream_t st) {
  if (!status || limit_ns == 0 || limit_ns > 1000000000ull) return TEMPLORA_ERR_INVALID_ARG;   // at most 1 s
  wait_selftest_kernel<<<1, 32, 0, st>>>(status, limit_ns, 900);
  TL_CUDA_CHECK(cudaGetLastError());
  return TEMPLORA_OK;
}

void tc_set_stream_sm_limit(cudaStream_t st, int max_sms) {
  std::lock_guard<std::mutex> lk(g_limit_mu);
  if (max_sms <= 0) g_stream_limit.erase(st); else g_stream_limit[st] = max_sms;
}

int tc_decode_cluster_count(int cluster_size, int n_tokens, cudaStream_t st) {
  DeviceInfo *di = device_info();
  if (!di || di->cc_major != 10 || n_tokens < 1 || n_tokens > 16) return 0;
  const bool big = dcl::stages_that_fit(cluster_size, 4, n_tokens) >= 3;
  int fit;
  if (cluster_size == 2) fit = big ? decode_cluster_fit<2, 4>(di, 0) : decode_cluster_fit<2, 2>(di, 1);
  else if (cluster_size == 4) fit = big ? decode_cluster_fit<4, 4>(di, 2) : decode_cluster_fit<4, 2>(di, 3);
  else return 0;
  const int cap = stream_sm_limit(st, di->sm_count) / cluster_size;
  if (fit > cap) fit = cap;
  return fit < 0 ? 0 : fit;
}

bool tc_available() {
  DeviceInfo *di = device_info();
  return di && di->cc_major == 10 && encode_fn() != nullptr;
}

templora_status_t tc_gemm_grouped(const TcProblem *probs, int n, int BN, DeviceStatus *status, cudaStream_t st,
                                  int cta_pairs, int order_mode) {
  if (n <= 0 || n > kTcMaxProblems) return TEMPLORA_ERR_INVALID_ARG;
  const bool use_pair = cta_pairs && BN == 256;   // 256 x 256 tiles on CTA pairs
  const int tile_m = use_pair ? 256 : BM;         // rows of one work item
  const int box_b = use_pair ? 128 : BN;          // rows of the B-operand box one CTA loads
  if (BN != 16 && BN != 64 && BN != 256) return TEMPLORA_ERR_INVALID_ARG;
  DeviceInfo *di = device_info();
  if (!di || di->cc_major != 10) return TEMPLORA_ERR_UNSUPPORTED;
  if (!status) return TEMPLORA_ERR_WORKSPACE;  // the kernel keeps its item counter in the status record

  // heaviest work items first: the static round-robin schedule then ends on the short ones
  int order[kTcMaxProblems];
  for (int i = 0; i < n; ++i) order[i] = order_mode == 2 ? n - 1 - i : i;
  auto weight = [&](int i) {
    const TcProblem &p = probs[i];
    long long kb = (p.K + BK - 1) / BK;
    int s = p.splits < 1 ? 1 : p.splits;
    long long w = (kb + s - 1) / s + (p.Kext + BK - 1) / BK;
    for (int e = 0; e < p.n_extra; ++e) w += (p.Kx[e] + BK - 1) / BK;
    if (p.epi_mode == 1) w += (p.Kext + BK - 1) / BK;
    return w;
  };
  for (int i = 1; i < n && order_mode == 0; ++i)
    for (int j = i; j > 0 && weight(order[j]) > weight(order[j - 1]); --j) {
      int t = order[j]; order[j] = order[j - 1]; order[j - 1] = t;
    }

  DevGroup g;
  g.status = status;
  g.n_prob = n;
  int items = 0;
  for (int i = 0; i < n; ++i) {
    const TcProblem &p = probs[order[i]];
    DevProb &q = g.p[i];
    if (p.M <= 0 || p.N <= 0 || p.K <= 0 || p.Kext < 0 || !p.A || !p.B || !p.out) return TEMPLORA_ERR_INVALID_ARG;
    if (p.b_mn && BN < 64) return TEMPLORA_ERR_UNSUPPORTED;
    if ((p.lda | p.ldb) & 7) return TEMPLORA_ERR_UNSUPPORTED;
    q.M = p.M; q.N = p.N;
    q.kb_main = (p.K + BK - 1) / BK;
    q.kb_ext = (p.Kext + BK - 1) / BK;
    q.splits = p.splits < 1 ? 1 : (p.splits > q.kb_main ? q.kb_main : p.splits);
    if (use_pair && (p.splits > 1 || p.out_f32 || p.out_s1 != 1 || p.epi_mask || (p.out_s0 & 7) ||
                     (reinterpret_cast<uintptr_t>(p.out) & 15)))
      return TEMPLORA_ERR_UNSUPPORTED;   // the pair kernel writes bf16 rows through bulk tensor stores
    q.m_tiles = (p.M + tile_m - 1) / tile_m;
    q.n_tiles = (p.N + BN - 1) / BN;
    q.epi_mode = p.epi_mode; q.pad4 = 0;
    q.epi_in0 = reinterpret_cast<const __nv_bfloat16 *>(p.epi_in0);
    q.epi_in1 = reinterpret_cast<const __nv_bfloat16 *>(p.epi_in1);
    if (p.epi_mode != 0) {
      if (!use_pair || p.epi_mode < 0 || p.epi_mode > 2 || p.n_extra != 0 || !p.out1) return TEMPLORA_ERR_UNSUPPORTED;
      if (p.epi_mode == 1) {
        if (p.a_mn || p.b_mn || p.Kext <= 0 || !p.B1 || !p.Bext1 || !p.Aext1 || !p.out2 ||
            ((p.ldb1 | p.ldbext1 | p.ldaext1) & 7))
          return TEMPLORA_ERR_INVALID_ARG;
        q.n_tiles = (p.N + 127) / 128;   // a tile holds 128 columns of gate and the same 128 columns of up
      } else if (!p.epi_in0 || !p.epi_in1 || ((reinterpret_cast<uintptr_t>(p.epi_in0) | reinterpret_cast<uintptr_t>(p.epi_in1)) & 15)) {
        return TEMPLORA_ERR_INVALID_ARG;
      }
    }
    q.item_start = items;
    q.a_mn = p.a_mn; q.b_mn = p.b_mn;
    q.out_f32 = p.out_f32; q.pad = 0;
    q.epi_mask = p.epi_mask; q.epi_mask_pitch = p.epi_mask_pitch; q.epi_scale = p.epi_scale; q.pad3 = 0;
    if (p.epi_mask && (p.out_f32 || p.out_s1 != 1 || BN < 32)) return TEMPLORA_ERR_UNSUPPORTED;
    q.out = p.out; q.out_s0 = p.out_s0; q.out_s1 = p.out_s1; q.out_split = p.out_split;
    long long cnt = (long long)q.m_tiles * q.n_tiles * q.splits;
    if (cnt + items > 0x3fffffff) return TEMPLORA_ERR_UNSUPPORTED;
    items += (int)cnt;
    bool ok = make_operand_map(&q.tmA, p.A, p.M, p.K, p.lda, p.a_mn, BM) &&
              make_operand_map(&q.tmB, p.B, p.N, p.K, p.ldb, p.b_mn, box_b);
    if (p.Kext > 0) {
      if (!p.Aext || !p.Bext || ((p.ldaext | p.ldbext) & 7)) return TEMPLORA_ERR_INVALID_ARG;
      ok = ok && make_operand_map(&q.tmAe, p.Aext, p.M, p.Kext, p.ldaext, p.a_mn, BM) &&
           make_operand_map(&q.tmBe, p.Bext, p.N, p.Kext, p.ldbext, p.b_mn, box_b);
    } else {
      q.tmAe = q.tmA;
      q.tmBe = q.tmB;
    }
    q.kb_xtot = 0;
    if (p.n_extra < 0 || p.n_extra > kMaxExtra || (p.n_extra > 0 && q.splits > 1)) return TEMPLORA_ERR_INVALID_ARG;
    for (int e = 0; e < kMaxExtra; ++e) {
      q.kb_x[e] = 0;
      q.tmXa[e] = q.tmA;
      q.tmXb[e] = q.tmB;
      if (e >= p.n_extra) continue;
      if (!p.Ax[e] || !p.Bx[e] || p.Kx[e] <= 0 || ((p.ldax[e] | p.ldbx[e]) & 7)) return TEMPLORA_ERR_INVALID_ARG;
      q.kb_x[e] = (p.Kx[e] + BK - 1) / BK;
      q.kb_xtot += q.kb_x[e];
      ok = ok && make_operand_map(&q.tmXa[e], p.Ax[e], p.M, p.Kx[e], p.ldax[e], p.a_mn, BM) &&
           make_operand_map(&q.tmXb[e], p.Bx[e], p.N, p.Kx[e], p.ldbx[e], p.b_mn, box_b);
    }
    if (use_pair && p.epi_mode == 0) ok = ok && make_map(&q.tmOut, p.out, p.N, p.M, p.out_s0, 32);
    else q.tmOut = q.tmA;
    if (p.epi_mode != 0) {
      if ((reinterpret_cast<uintptr_t>(p.out1) & 15) || (p.out2 && (reinterpret_cast<uintptr_t>(p.out2) & 15)))
        return TEMPLORA_ERR_INVALID_ARG;
      ok = ok && make_map(&q.tmOut, p.out, p.N, p.M, p.out_s0, 32, 32) &&
           make_map(&q.tmXa[1], p.out1, p.N, p.M, p.out_s0, 32, 32);
      if (p.epi_mode == 1) {
        q.kb_x[0] = q.kb_ext;
        q.kb_xtot = q.kb_ext;
        ok = ok && make_map(&q.tmXa[2], p.out2, p.N, p.M, p.out_s0, 32, 32) &&
             make_operand_map(&q.tmXb[1], p.B1, p.N, p.K, p.ldb1, 0, box_b) &&
             make_operand_map(&q.tmXa[0], p.Aext1, p.M, p.Kext, p.ldaext1, 0, BM) &&
             make_operand_map(&q.tmXb[0], p.Bext1, p.N, p.Kext, p.ldbext1, 0, box_b);
      }
    }
    if (!ok) return TEMPLORA_ERR_CUDA;
  }
  g.n_items = items;
  static_assert(sizeof(DevGroup) <= 32000, "the launch description travels as a kernel parameter");
  if (use_pair) return launch_pair(g, di, st);
  if (BN == 256) return launch<256>(g, di, 0, st);
  if (BN == 64) return launch<64>(g, di, 1, st);
  return launch<16>(g, di, 2, st);
}

// Decode-time forward of up to dcl::kDclMaxProj projections in one launch.  probs holds, for each
// projection, its u problem (role 1) and its y problem (role 0, with the rank-r extension reading the
// u problem's output); flag is the projection's index.  The u problems must come first.
templora_status_t tc_decode_cluster(const TcProblem *probs, int n, int n_tokens, int cluster_size, DeviceStatus *status,
                                    cudaStream_t st) {
  if (n <= 0 || n > kTcMaxProblems || n_tokens < 1 || n_tokens > 16) return TEMPLORA_ERR_INVALID_ARG;
  DeviceInfo *di = device_info();
  if (!di || di->cc_major != 10) return TEMPLORA_ERR_UNSUPPORTED;
  if (!status) return TEMPLORA_ERR_WORKSPACE;
  DevGroup g;
  g.status = status;
  g.n_prob = n;
  int items = 0, n_u = 0;
  for (int i = 0; i < n; ++i) {
    const TcProblem &p = probs[i];
    DevProb &q = g.p[i];
    if (p.M <= 0 || p.N != n_tokens || p.K <= 0 || p.Kext < 0 || !p.A || !p.B || !p.out) return TEMPLORA_ERR_INVALID_ARG;
    if (p.a_mn || p.b_mn || p.out_f32 || p.out_s0 != 1 || ((p.lda | p.ldb) & 7)) return TEMPLORA_ERR_UNSUPPORTED;
    if (p.flag < 0 || p.flag >= dcl::kDclMaxProj) return TEMPLORA_ERR_INVALID_ARG;
    if (p.role == 1) {
      if (n_u != i || p.Kext != 0) return TEMPLORA_ERR_INVALID_ARG;   // u problems first, no extension
      ++n_u;
    }
    q.M = p.M; q.N = p.N;
    q.kb_main = (p.K + BK - 1) / BK;
    q.kb_ext = (p.Kext + BK - 1) / BK;
    q.splits = 1;
    q.m_tiles = (p.M + BM - 1) / BM;
    q.n_tiles = 1;
    q.item_start = items;
    q.a_mn = 0; q.b_mn = 0; q.out_f32 = 0;
    q.pad = p.role; q.pad3 = p.flag;
    q.kb_xtot = 0;
    for (int e = 0; e < kMaxExtra; ++e) { q.kb_x[e] = 0; q.tmXa[e] = q.tmA; q.tmXb[e] = q.tmB; }
    q.tmOut = q.tmA;
    q.epi_mode = 0; q.pad4 = 0; q.epi_in0 = nullptr; q.epi_in1 = nullptr;
    q.epi_mask = nullptr; q.epi_mask_pitch = 0; q.epi_scale = p.epi_scale;
    q.out = p.out; q.out_s0 = 1; q.out_s1 = p.out_s1; q.out_split = 0;
    items += q.m_tiles;
    bool ok = make_operand_map(&q.tmA, p.A, p.M, p.K, p.lda, 0, BM) && make_operand_map(&q.tmB, p.B, p.N, p.K, p.ldb, 0, 16);
    if (p.Kext > 0) {
      if (!p.Aext || !p.Bext || ((p.ldaext | p.ldbext) & 7)) return TEMPLORA_ERR_INVALID_ARG;
      ok = ok && make_operand_map(&q.tmAe, p.Aext, p.M, p.Kext, p.ldaext, 0, BM) &&
           make_operand_map(&q.tmBe, p.Bext, p.N, p.Kext, p.ldbext, 0, 16);
    } else {
      q.tmAe = q.tmA;
      q.tmBe = q.tmB;
    }
    if (!ok) return TEMPLORA_ERR_CUDA;
  }
  g.n_items = items;
  dcl::DclParams prm;
  prm.n_tokens = n_tokens;
  // every u item must be the first item of its cluster (it then waits for nothing): the launchers
  // below start cluster c on item c, so they need at least n_u clusters
  // 72 KB stages (four k-blocks) when three of them fit beside the receive buffer, else 36 KB stages
  const bool big = dcl::stages_that_fit(cluster_size, 4, n_tokens) >= 3;
  templora_status_t rc;
  if (cluster_size == 2)
    rc = big ? launch_decode_cluster<2, 4>(g, prm, di, 0, st, n_u) : launch_decode_cluster<2, 2>(g, prm, di, 1, st, n_u);
  else if (cluster_size == 4)
    rc = big ? launch_decode_cluster<4, 4>(g, prm, di, 2, st, n_u) : launch_decode_cluster<4, 2>(g, prm, di, 3, st, n_u);
  else
    return TEMPLORA_ERR_INVALID_ARG;
  return rc;
}

}  // namespace templora
