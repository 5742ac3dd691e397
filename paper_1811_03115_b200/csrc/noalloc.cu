// bpd_op_vocab_argmax_noalloc: the vocabulary top-1 for callers that cannot
// provide (or allocate) a workspace.  The cross-CTA reduction workspace lives
// in a fixed device array that is part of this library's image.
#include <mutex>

#include "host.hpp"
#include "kernels_simt.cuh"

namespace bpd {

constexpr int kNoAllocMaxRows = 256;
constexpr int kNoAllocMaxVocab = 65536;
constexpr int kNoAllocMaxTiles = kNoAllocMaxVocab / kVocTile;
constexpr size_t kNoAllocValBytes = (size_t)kNoAllocMaxTiles * kNoAllocMaxRows * sizeof(float);
constexpr size_t kNoAllocIdxBytes = (size_t)kNoAllocMaxTiles * kNoAllocMaxRows * sizeof(int);
constexpr size_t kNoAllocCntBytes = 256;   // one counter per group of kRC rows: 32 of them, padded
constexpr size_t kNoAllocBytes = kNoAllocValBytes + kNoAllocIdxBytes + kNoAllocCntBytes;

// 512 KiB + 256 B of global memory on every GPU that loads this library, held until the process exits.
// In host code this name is only a handle for the runtime, not a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_noalloc_mutex;
static unsigned char* g_noalloc_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the current device, looked up once per device.
static int noalloc_scratch(unsigned char** out) {
  int dev = -1;
  BPD_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(BPD_E_UNSUPPORTED, "device ordinal %d above %d", dev, kMaxDevices - 1);
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p)
      return fail(BPD_E_CUDA, "cudaGetSymbolAddress(static scratch) failed on device %d: %s", dev, cudaGetErrorString(e));
    g_noalloc_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_noalloc_ptr[dev];
  return BPD_OK;
}

}  // namespace bpd

using namespace bpd;

extern "C" int bpd_op_vocab_argmax_noalloc(const void* x, const void* w, int rows, int d, int vocab, int dtype,
                                           int32_t* out_idx, float* out_val, void* cuda_stream) {
  if (!x || !w || !out_idx) return fail(BPD_E_INVALID, "null argument");
  if (dtype != 0 && dtype != 1) return fail(BPD_E_INVALID, "unknown dtype %d", dtype);
  if (rows < 1 || vocab < 1 || d < 8 || d % 8 || d > kArgmaxMaxD)
    return fail(BPD_E_SHAPE, "rows/d/vocab out of range (d must be a multiple of 8, at most %d)", kArgmaxMaxD);
  if (rows > kNoAllocMaxRows || vocab > kNoAllocMaxVocab)
    return fail(BPD_E_NOMEM, "rows = %d, vocab = %d exceed the built-in workspace (at most %d rows, vocabulary %d); "
                "use bpd_op_vocab_argmax with a caller-provided scratch buffer", rows, vocab, kNoAllocMaxRows, kNoAllocMaxVocab);
  if ((uintptr_t)x % 16 || (uintptr_t)w % 16) return fail(BPD_E_INVALID, "misaligned pointer");
  unsigned char* base = nullptr;
  int rc = noalloc_scratch(&base);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  float* part_val = reinterpret_cast<float*>(base);
  int* part_idx = reinterpret_cast<int*>(base + kNoAllocValBytes);
  unsigned* counters = reinterpret_cast<unsigned*>(base + kNoAllocValBytes + kNoAllocIdxBytes);
  // the array keeps whatever the previous call left: the arrival counters must start at zero
  BPD_CUDA(cudaMemsetAsync(counters, 0, kNoAllocCntBytes, st));
  ArgmaxParams p{x, (long long)d, w, rows, d, vocab, part_val, part_idx, counters, out_idx, out_val, nullptr, nullptr};
  dim3 grid((vocab + kVocTile - 1) / kVocTile, (rows + kRC - 1) / kRC);
  const size_t smem = (size_t)kRC * d * sizeof(float);
  if (dtype == 0) vocab_argmax_kernel<float, float><<<grid, kLinWarps * 32, smem, st>>>(p);
  else vocab_argmax_kernel<bf16, bf16><<<grid, kLinWarps * 32, smem, st>>>(p);
  ++g_launches;
  BPD_CUDA(cudaGetLastError());
  return BPD_OK;
}
