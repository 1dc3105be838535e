// bild_op_lm_head_static: the fused LM head without any caller-provided scratch.
//
// Some users of this library cannot hand it scratch memory because they cannot allocate
// any: a decode worker running inside a serving process whose own allocator has already
// claimed the device's memory, or a latency-critical loop that must not call cudaMalloc
// because that call synchronises the whole device and stalls the other streams.  For
// them the block partials, the ticket counter and the result record of the LM-head kernel
// live in one fixed array in this library's device image.
#include <cstdio>
#include <mutex>

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bild.h"

namespace {  // this file's own instance of the kernel templates (internal linkage)
#include "kernels.cuh"
}  // namespace

using namespace bild;

namespace {

constexpr int STATIC_HEAD_GRID_MAX = 148 * 4;     // same block-count cap as the regular entry point
constexpr size_t STATIC_SCRATCH_BYTES = 128 * 1024;
constexpr int STATIC_MAX_V = 1 << 20;
constexpr int STATIC_MAX_K = 4096;
constexpr int MAX_DEVICES = 64;

// Lives in every GPU that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_static_head_scratch[STATIC_SCRATCH_BYTES];

std::mutex g_mu;
void* g_dev_ptr[MAX_DEVICES];   // device address of the array, per device ordinal

size_t up256(size_t v) { return (v + 255) / 256 * 256; }
int grid_for(int V) { return V < 64 ? 1 : (V + 63) / 64 > STATIC_HEAD_GRID_MAX ? STATIC_HEAD_GRID_MAX : (V + 63) / 64; }

// In host code the array's name is only a handle; the address kernels can use comes from
// the runtime, once per device, with that device current.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return BILD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_dev_ptr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_head_scratch);
    if (e != cudaSuccess || !p) {
      std::fprintf(stderr, "bild_op_lm_head_static: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
      return BILD_ERR_CUDA;
    }
    g_dev_ptr[dev] = p;
  }
  *out = g_dev_ptr[dev];
  return BILD_OK;
}

// *too_big: the MB staged rows of K floats plus the kernel's own shared memory exceed what a block may have
template <typename WT, int MB, int RW>
cudaError_t launch_t(const HeadArgs& a, int grid, cudaStream_t s, bool* too_big) {
  const size_t smem = (size_t)MB * a.K * sizeof(float);
  auto kern = lm_head_kernel<WT, MB, RW>;
  if (smem > 48 * 1024) {
    cudaFuncAttributes fa;
    int dev = 0, optin = 0;
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e == cudaSuccess) e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return e;
    if (smem + fa.sharedSizeBytes > (size_t)optin) { *too_big = true; return cudaSuccess; }
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  kern<<<grid, HEAD_THREADS, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace

extern "C" int bild_op_lm_head_static(const void* W, int w_dtype, const float* X, const float* gain, float eps,
                                      float scale, const int32_t* target, int M, int V, int K, int32_t* argmax_out,
                                      float* max_out, float* lse_out, float* gather_out, void* cuda_stream) {
  if (!W || !X || !argmax_out || !max_out || !lse_out) return BILD_ERR_ARG;
  if (w_dtype != BILD_FP32 && w_dtype != BILD_BF16) return BILD_ERR_ARG;
  if (M < 1 || V < 1 || K < 8 || K % 8) return BILD_ERR_ARG;
  if (M > MAXB || V > STATIC_MAX_V || K > STATIC_MAX_K) {
    std::fprintf(stderr, "bild_op_lm_head_static: M=%d V=%d K=%d exceeds the built-in scratch (M <= %d, V <= %d, "
                 "K <= %d); use bild_op_lm_head with caller scratch\n", M, V, K, MAXB, STATIC_MAX_V, STATIC_MAX_K);
    return BILD_ERR_CAPACITY;
  }
  const int grid = grid_for(V);
  const size_t need = up256((size_t)grid * MAXB * sizeof(Partial)) + 256 + up256(sizeof(HeadOut));
  if (need > STATIC_SCRATCH_BYTES) {
    std::fprintf(stderr, "bild_op_lm_head_static: needs %zu bytes of scratch, the built-in array has %zu\n", need,
                 STATIC_SCRATCH_BYTES);
    return BILD_ERR_CAPACITY;
  }
  void* base = nullptr;
  int rc = scratch_for_current_device(&base);
  if (rc != BILD_OK) return rc;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  char* p = (char*)base;
  HeadArgs h{};
  h.partials = (Partial*)p;
  p += up256((size_t)grid * MAXB * sizeof(Partial));
  h.counter = (unsigned*)p;
  p += 256;
  h.out = (HeadOut*)p;
  // the array keeps whatever the previous call left: the ticket counter must start at zero
  if (cudaMemsetAsync(h.counter, 0, sizeof(unsigned), s) != cudaSuccess) return BILD_ERR_CUDA;
  if (cudaMemsetAsync(h.out, 0, sizeof(HeadOut), s) != cudaSuccess) return BILD_ERR_CUDA;
  h.W = W; h.X = X; h.ldx = K; h.gain = gain; h.eps = eps; h.scale = scale; h.V = V; h.K = K; h.M = M;
  h.target = target; h.logits_dbg = nullptr; h.which = 1;
  cudaError_t e;
  bool too_big = false;
  const int MB = M == 1 ? 1 : MAXB;
  if (w_dtype == BILD_BF16)
    e = MB == 1 ? launch_t<__nv_bfloat16, 1, 4>(h, grid, s, &too_big) : launch_t<__nv_bfloat16, MAXB, 2>(h, grid, s, &too_big);
  else
    e = MB == 1 ? launch_t<float, 1, 4>(h, grid, s, &too_big) : launch_t<float, MAXB, 2>(h, grid, s, &too_big);
  if (too_big) {
    std::fprintf(stderr, "bild_op_lm_head_static: %d staged rows of K=%d floats do not fit a block's shared memory "
                 "(M >= 2 takes K <= about 3500)\n", MB, K);
    return BILD_ERR_CAPACITY;
  }
  if (e != cudaSuccess) return BILD_ERR_CUDA;
  const HeadOut* o = h.out;
  e = cudaMemcpyAsync(argmax_out, o->argmax, M * sizeof(int), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(max_out, o->zmax, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(lse_out, o->lse, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess && gather_out && target)
    e = cudaMemcpyAsync(gather_out, o->gather, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  return e == cudaSuccess ? BILD_OK : BILD_ERR_CUDA;
}
