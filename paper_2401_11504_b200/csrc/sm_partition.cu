// SM partitions for the parallelized deployment: the chunk update and the decode stream side by side on one GPU.
//
// A per-stream cap on the persistent kernels' grid sizes (templora_set_stream_sm_limit) bounds how many SMs
// each side asks for, but not WHICH ones: every time the update stream starts its next kernel its CTAs take
// whatever SMs happen to be free, and the decode kernel's CTA pairs (clusters of two: both SMs of one TPC) then
// wait until a whole TPC has drained.  Here the two sides get disjoint sets of SMs instead: the device's SMs
// are split into two groups, each group backs a green context, and a stream created in a green context only
// ever runs kernels on its group.  The first group is sized by the caller (rounded by the driver to its
// granularity, 8 SMs on this architecture), the second gets the rest.
//
// The driver entry points are looked up at run time, so the library keeps loading on a machine without a GPU.
#include "common.cuh"

#include <cuda.h>

#include <new>

namespace templora {
namespace {

template <typename F> F driver_fn(const char *name) {
  void *p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) return nullptr;
  return reinterpret_cast<F>(p);
}

typedef CUresult (*DeviceGetFn)(CUdevice *, int);
typedef CUresult (*GetDevResourceFn)(CUdevice, CUdevResource *, CUdevResourceType);
typedef CUresult (*SplitByCountFn)(CUdevResource *, unsigned int *, const CUdevResource *, CUdevResource *, unsigned int,
                                   unsigned int);
typedef CUresult (*GenerateDescFn)(CUdevResourceDesc *, CUdevResource *, unsigned int);
typedef CUresult (*GreenCtxCreateFn)(CUgreenCtx *, CUdevResourceDesc, CUdevice, unsigned int);
typedef CUresult (*GreenCtxDestroyFn)(CUgreenCtx);
typedef CUresult (*GreenCtxStreamCreateFn)(CUstream *, CUgreenCtx, unsigned int, int);
typedef CUresult (*StreamDestroyFn)(CUstream);

struct Partition {
  CUgreenCtx ctx[2] = {nullptr, nullptr};
  CUstream stream[2] = {nullptr, nullptr};
  int sms[2] = {0, 0};
};

void destroy(Partition *p) {
  auto stream_destroy = driver_fn<StreamDestroyFn>("cuStreamDestroy");
  auto ctx_destroy = driver_fn<GreenCtxDestroyFn>("cuGreenCtxDestroy");
  for (int i = 0; i < 2; ++i) {
    if (p->stream[i]) {
      tc_set_stream_sm_limit(reinterpret_cast<cudaStream_t>(p->stream[i]), 0);
      if (stream_destroy) stream_destroy(p->stream[i]);
    }
    if (p->ctx[i] && ctx_destroy) ctx_destroy(p->ctx[i]);
  }
  delete p;
}

}  // namespace
}  // namespace templora

using namespace templora;

extern "C" templora_status_t templora_sm_partition_create(int32_t first_sms, templora_sm_partition_t *out) {
  if (!out || first_sms < 1) return TEMPLORA_ERR_INVALID_ARG;
  out->handle = nullptr;
  out->stream_first = out->stream_rest = nullptr;
  out->sms_first = out->sms_rest = 0;
  auto device_get = driver_fn<DeviceGetFn>("cuDeviceGet");
  auto get_resource = driver_fn<GetDevResourceFn>("cuDeviceGetDevResource");
  auto split = driver_fn<SplitByCountFn>("cuDevSmResourceSplitByCount");
  auto gen_desc = driver_fn<GenerateDescFn>("cuDevResourceGenerateDesc");
  auto ctx_create = driver_fn<GreenCtxCreateFn>("cuGreenCtxCreate");
  auto stream_create = driver_fn<GreenCtxStreamCreateFn>("cuGreenCtxStreamCreate");
  if (!device_get || !get_resource || !split || !gen_desc || !ctx_create || !stream_create) return TEMPLORA_ERR_UNSUPPORTED;

  int ordinal = 0;
  TL_CUDA_CHECK(cudaGetDevice(&ordinal));
  TL_CUDA_CHECK(cudaFree(nullptr));   // the device's primary context exists from here on
  CUdevice dev;
  if (device_get(&dev, ordinal) != CUDA_SUCCESS) return TEMPLORA_ERR_CUDA;
  CUdevResource all, group[2];
  if (get_resource(dev, &all, CU_DEV_RESOURCE_TYPE_SM) != CUDA_SUCCESS) return TEMPLORA_ERR_UNSUPPORTED;
  if ((unsigned)first_sms >= all.sm.smCount) return TEMPLORA_ERR_INVALID_ARG;
  unsigned int n_groups = 1;
  if (split(&group[0], &n_groups, &all, &group[1], 0, (unsigned)first_sms) != CUDA_SUCCESS || n_groups != 1)
    return TEMPLORA_ERR_UNSUPPORTED;
  if (group[1].sm.smCount == 0) return TEMPLORA_ERR_INVALID_ARG;   // rounding left nothing for the other side

  Partition *p = new (std::nothrow) Partition;
  if (!p) return TEMPLORA_ERR_CUDA;
  for (int i = 0; i < 2; ++i) {
    CUdevResourceDesc desc;
    if (gen_desc(&desc, &group[i], 1) != CUDA_SUCCESS || ctx_create(&p->ctx[i], desc, dev, CU_GREEN_CTX_DEFAULT_STREAM) != CUDA_SUCCESS ||
        stream_create(&p->stream[i], p->ctx[i], CU_STREAM_NON_BLOCKING, 0) != CUDA_SUCCESS) {
      destroy(p);
      return TEMPLORA_ERR_UNSUPPORTED;
    }
    p->sms[i] = (int)group[i].sm.smCount;
    // the persistent kernels size their grids by this figure
    tc_set_stream_sm_limit(reinterpret_cast<cudaStream_t>(p->stream[i]), p->sms[i]);
  }
  out->handle = p;
  out->stream_first = p->stream[0];
  out->stream_rest = p->stream[1];
  out->sms_first = p->sms[0];
  out->sms_rest = p->sms[1];
  return TEMPLORA_OK;
}

extern "C" templora_status_t templora_sm_partition_destroy(templora_sm_partition_t *part) {
  if (!part || !part->handle) return TEMPLORA_ERR_INVALID_ARG;
  Partition *p = reinterpret_cast<Partition *>(part->handle);
  for (int i = 0; i < 2; ++i)
    if (p->stream[i] && cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(p->stream[i])) != cudaSuccess) return TEMPLORA_ERR_CUDA;
  destroy(p);
  part->handle = nullptr;
  part->stream_first = part->stream_rest = nullptr;
  part->sms_first = part->sms_rest = 0;
  return TEMPLORA_OK;
}
