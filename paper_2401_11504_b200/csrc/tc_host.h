// Host-side helpers shared by the tensor-core kernels' launchers: tensor-map encoding (cached per thread),
// per-device facts and the per-stream SM cap.  Defined in tc_gemm.cu.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace templora {

// 2-D bf16 tensor [outer][inner] with row pitch `pitch` elements; box = box_inner x box_outer elements
// (box_inner 64: 128-byte swizzle; 32: not swizzled).  False when the driver refuses the description.
bool make_map(CUtensorMap *m, const void *ptr, long long inner, long long outer, long long pitch, int box_outer,
              int box_inner = 64);
// MMA operand [rows = M or N][K] (mn = 0: boxes of tile_mn rows x 64 k) or [K][M or N] (mn = 1: boxes of 64 x 64)
bool make_operand_map(CUtensorMap *m, const void *ptr, long long mn_extent, long long k_extent, long long ld, int mn,
                      int tile_mn);

struct DeviceInfo {
  int sm_count = 0;
  int cc_major = 0;
  bool attr_set[3] = {false, false, false};
  bool pair_attr_set = false;
  int dcl_clusters[4] = {};   // per decode-cluster kernel variant: clusters that fit at once (0 = not asked yet, -1 = none)
};
DeviceInfo *device_info();   // of the current device; nullptr when it cannot be queried

// SMs the persistent kernels may occupy on this stream (templora_set_stream_sm_limit), at most sm_count
int stream_sm_limit(cudaStream_t st, int sm_count);

}  // namespace templora
