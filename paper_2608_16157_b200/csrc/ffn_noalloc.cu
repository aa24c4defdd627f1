// ft_moe_ffn_noalloc: the streaming SwiGLU expert FFN for callers that must not allocate.
//
// The regular path keeps its scratch (the fp32 output accumulator, the work list and the CTA
// completion counter) in memory that ft_moe_create obtained with cudaMalloc.  Some callers cannot do
// that: code running inside a region where the allocator is off limits (a real-time serving loop
// with a frozen memory budget, a plug-in loaded into a process whose memory pool is owned by someone
// else, a library initialised after the application has claimed all of HBM).  For them this file
// keeps the scratch in a fixed array in the module's own device data segment.  Every GPU that loads
// the library holds that array until the process exits.
#include "../../include/ftmoe.h"

#include <cuda_runtime.h>

#include <cstddef>
#include <mutex>

#include "ffn_stream.cuh"

using namespace ftmoe;

namespace {

constexpr int kNoAllocMaxTokens = FT_NOALLOC_MAX_TOKENS;
constexpr int kNoAllocMaxHidden = FT_NOALLOC_MAX_HIDDEN;
constexpr size_t kAccBytes = (size_t)kNoAllocMaxTokens * kNoAllocMaxHidden * sizeof(float);
constexpr size_t kCtlBytes = 256;  // work item, pass prefix, item count, completion counter, status
constexpr size_t kScratchBytes = kAccBytes + kCtlBytes;

// Layout: [0, kAccBytes) fp32 accumulator [T][hidden]; then the control block below.
struct NoAllocCtl {
  WorkItem item;       // the one expert: all T tokens, gate weight 1
  int32_t pref[2];     // {0, passes}
  int32_t n_items;     // 1
  int32_t n_zc;        // 0: no host-resident records here
  uint32_t done;       // CTA completion counter of the kernel
  uint32_t status;     // latched device status, read and cleared by ft_moe_ffn_noalloc_status
};
static_assert(sizeof(NoAllocCtl) <= kCtlBytes, "control block too large");

// In host code this name is only a handle for cudaGetSymbolAddress; device code may use it directly.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// Clears the part of the accumulator this call uses and writes the control block.  Runs on the
// caller's stream right before the FFN kernel, so the previous call's leftovers never leak in.
__global__ void noalloc_setup_kernel(const uint8_t *record, int T, int hidden) {
  float4 *acc = reinterpret_cast<float4 *>(g_noalloc_scratch);
  const int n4 = T * hidden / 4;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x)
    acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    NoAllocCtl *ctl = reinterpret_cast<NoAllocCtl *>(g_noalloc_scratch + kAccBytes);
    ctl->item.w = record;
    ctl->item.expert = -1;   // tokens 0..T-1, weight 1
    ctl->item.n_tok = T;
    ctl->item.off = 0;
    ctl->item.slot = -1;
    ctl->pref[0] = 0;
    ctl->pref[1] = (T + kFsResTokensPerPass - 1) / kFsResTokensPerPass;
    ctl->n_items = 1;
    ctl->n_zc = 0;
    ctl->done = 0u;
    // ctl->status stays latched until ft_moe_ffn_noalloc_status reads and clears it
  }
}

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;                               // guards the two tables below
unsigned char *g_scratch_ptr[kMaxDevices] = {nullptr};  // device address of the array, per device
int g_sm_count[kMaxDevices] = {0};

// Restores the calling thread's current device when the entry point returns.
struct DeviceGuard {
  int prev = -1;
  DeviceGuard() { if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; (void)cudaGetLastError(); } }
  ~DeviceGuard() { if (prev >= 0) (void)cudaSetDevice(prev); }
};

// Once per device, with that device current: resolve the array's device address and raise the
// kernels' dynamic shared memory limit.  Neither call allocates.
ft_status_t noalloc_setup_device(int dev) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[dev] != nullptr) return FT_OK;
  unsigned char *ptr = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
    (void)cudaGetLastError();
    return FT_ERR_CUDA;
  }
  const int smem = (int)ffn_stream_smem_bytes(1, kNoAllocMaxHidden);
  if (cudaFuncSetAttribute(ffn_stream_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaFuncSetAttribute(ffn_stream_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaFuncSetAttribute(ffn_stream_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaFuncSetAttribute(ffn_stream_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
    (void)cudaGetLastError();
    return FT_ERR_CUDA;
  }
  int smc = 0;
  if (cudaDeviceGetAttribute(&smc, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || smc <= 0) {
    (void)cudaGetLastError();
    return FT_ERR_CUDA;
  }
  g_sm_count[dev] = smc;
  g_scratch_ptr[dev] = ptr;
  return FT_OK;
}

}  // namespace

extern "C" ft_status_t ft_moe_ffn_noalloc(int device, const void *record_dev, int hidden, int inter,
                                          const void *x_dev, void *y_dev, int T, void *stream) {
  if (device < 0 || device >= kMaxDevices || !record_dev || !x_dev || !y_dev) return FT_ERR_INVALID_ARG;
  if (T < 1 || T > kNoAllocMaxTokens) return FT_ERR_INVALID_ARG;       // beyond the static scratch
  if (hidden > kNoAllocMaxHidden) return FT_ERR_INVALID_ARG;           // beyond the static scratch
  if ((hidden != 256 && hidden != 512 && hidden != 1024 && hidden != 2048) || inter < 16 || inter % 16)
    return FT_ERR_UNSUPPORTED;
  // the kernel reads the record and x with 16-byte loads and writes y with 8-byte stores
  if (((uintptr_t)record_dev | (uintptr_t)x_dev | (uintptr_t)y_dev) & 15) return FT_ERR_INVALID_ARG;
  DeviceGuard guard;
  if (cudaSetDevice(device) != cudaSuccess) { (void)cudaGetLastError(); return FT_ERR_CUDA; }
  ft_status_t rc = noalloc_setup_device(device);
  if (rc != FT_OK) return rc;
  unsigned char *scratch;
  int grid;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    scratch = g_scratch_ptr[device];
    grid = g_sm_count[device];
  }
  NoAllocCtl *ctl = reinterpret_cast<NoAllocCtl *>(scratch + kAccBytes);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  noalloc_setup_kernel<<<32, 256, 0, st>>>(static_cast<const uint8_t *>(record_dev), T, hidden);

  FfnStreamParams mp;
  mp.items = &ctl->item;
  mp.n_items = &ctl->n_items;
  mp.n_zc = &ctl->n_zc;
  mp.n_hit = &ctl->n_zc;   // unused with part = 0
  mp.part = 0;
  mp.pref = ctl->pref;
  mp.max_items = 1;
  mp.trace = nullptr;
  mp.x = static_cast<const __nv_bfloat16 *>(x_dev);
  mp.perm = nullptr;       // unused: the item addresses tokens directly
  mp.topk_w = nullptr;
  mp.y_acc = reinterpret_cast<float *>(scratch);
  mp.y = static_cast<__nv_bfloat16 *>(y_dev);
  mp.done = &ctl->done;
  mp.status = &ctl->status;
  mp.inter = inter; mp.top_k = 1; mp.T = T; mp.finalize = 1; mp.overlap = 0;
  const size_t smem = ffn_stream_smem_bytes(1, hidden);
  switch (hidden / 256) {
    case 1: ffn_stream_kernel<1><<<grid, kFsThreads, smem, st>>>(mp); break;
    case 2: ffn_stream_kernel<2><<<grid, kFsThreads, smem, st>>>(mp); break;
    case 4: ffn_stream_kernel<4><<<grid, kFsThreads, smem, st>>>(mp); break;
    default: ffn_stream_kernel<8><<<grid, kFsThreads, smem, st>>>(mp); break;
  }
  if (cudaGetLastError() != cudaSuccess) return FT_ERR_CUDA;
  return FT_OK;
}

extern "C" ft_status_t ft_moe_ffn_noalloc_status(int device) {
  if (device < 0 || device >= kMaxDevices) return FT_ERR_INVALID_ARG;
  DeviceGuard guard;
  if (cudaSetDevice(device) != cudaSuccess) { (void)cudaGetLastError(); return FT_ERR_CUDA; }
  if (cudaDeviceSynchronize() != cudaSuccess) { (void)cudaGetLastError(); return FT_ERR_CUDA; }
  const size_t off = kAccBytes + offsetof(NoAllocCtl, status);
  uint32_t st = 0;
  if (cudaMemcpyFromSymbol(&st, g_noalloc_scratch, sizeof(st), off, cudaMemcpyDeviceToHost) != cudaSuccess) {
    (void)cudaGetLastError();
    return FT_ERR_CUDA;
  }
  if (st != 0) {
    const uint32_t zero = 0;
    if (cudaMemcpyToSymbol(g_noalloc_scratch, &zero, sizeof(zero), off, cudaMemcpyHostToDevice) != cudaSuccess) {
      (void)cudaGetLastError();
      return FT_ERR_CUDA;
    }
    return (st & kStatTimeout) ? FT_ERR_TIMEOUT : FT_ERR_CUDA;
  }
  return FT_OK;
}
