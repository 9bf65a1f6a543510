// cdgrab_step_noalloc: one balancing step for callers that must not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- inside a region whose
// memory is fully budgeted by a framework's caching allocator (a raw cudaMalloc there can
// fail or fragment the pool), inside latency-critical loops where the implicit device
// synchronisation of cudaMalloc/cudaFree is not acceptable, or in plug-ins that are handed
// buffers and a stream and nothing else.  Such callers keep r and the signs in their own
// buffers; the scratch the two-pass formulation needs (per-block partial sums, the Gram
// matrix, a few words of bookkeeping) lives in one fixed array in the library's device image.
//
// The array is shared by every call on a device and keeps what the last call left in it, so
// the words that must start at zero are cleared on the stream at every call, and two calls
// whose work overlaps on the GPU (different streams, no ordering) race on it.
#include <string.h>

#include "common.cuh"

namespace {

constexpr int kNaMaxM = 16;          // the register-resident FMA Gram kernels hold m <= 16
constexpr int kNaMaxBlocks = 512;    // partial vectors of at most 152 doubles each
constexpr int kNaMaxDevices = 64;

// byte offsets inside the scratch array
constexpr size_t kOffPartials = 0;
constexpr size_t kOffGram = kOffPartials + sizeof(double) * 152 * kNaMaxBlocks;
constexpr size_t kOffRnorm2 = kOffGram + sizeof(double) * (kNaMaxM * kNaMaxM + kNaMaxM);
constexpr size_t kOffStatus = kOffRnorm2 + sizeof(double);
constexpr size_t kOffPermCur = kOffStatus + 8;
constexpr size_t kOffPermNext = kOffPermCur + sizeof(int32_t) * 2 * kNaMaxM;
constexpr size_t kOffMargins = kOffPermNext + sizeof(int32_t) * 2 * kNaMaxM;
constexpr size_t kScratchBytes = ((kOffMargins + sizeof(float) * kNaMaxM + 255) / 256) * 256;

// 625,152 bytes held by every GPU that loads the library, until the process exits
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

struct NaDevice {
  unsigned char *scratch;  // device address of g_noalloc_scratch on this device
  int num_sms;
  int ready;
};
NaDevice g_na_dev[kNaMaxDevices];

// Once per device, with that device current: resolve the array's device address (in host code
// the symbol's name is only a stand-in, never a pointer a kernel could use) and fill the
// constant part of the scratch.  Synchronous.
int na_setup(int dev) {
  NaDevice &nd = g_na_dev[dev];
  if (nd.ready) return CDGRAB_OK;
  int major = 0, sms = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_DEVICE;
  }
  if (major != 10) return CDGRAB_ERR_DEVICE;
  unsigned char *ptr = nullptr;
  if (cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  // each worker's "current order" of its single pair is the identity (0, 1)
  int32_t ident[2 * kNaMaxM];
  for (int i = 0; i < kNaMaxM; ++i) { ident[2 * i] = 0; ident[2 * i + 1] = 1; }
  if (cudaMemcpy(ptr + kOffPermCur, ident, sizeof(ident), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  nd.scratch = ptr;
  nd.num_sms = sms;
  nd.ready = 1;
  return CDGRAB_OK;
}

}  // namespace

extern "C" int cdgrab_step_noalloc(int m, long long d, int dtype, const void *grads_dev, float *r_dev,
                                   int8_t *signs_out_dev, void *stream) {
  if (!grads_dev || !r_dev || !signs_out_dev) return CDGRAB_ERR_INVALID;
  if (dtype != CDGRAB_F32 && dtype != CDGRAB_BF16) return CDGRAB_ERR_INVALID;
  if (m < 1 || d < 4 || d % 4 != 0) return CDGRAB_ERR_INVALID;
  if (m > kNaMaxM) return CDGRAB_ERR_TOO_LARGE;  // the fixed scratch and kernels stop at 16 workers
  if (((uintptr_t)grads_dev & 15) != 0 || ((uintptr_t)r_dev & 15) != 0) return CDGRAB_ERR_INVALID;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_DEVICE; }
  if (dev < 0 || dev >= kNaMaxDevices) return CDGRAB_ERR_DEVICE;
  const int rc = na_setup(dev);
  if (rc != CDGRAB_OK) return rc;
  const NaDevice &nd = g_na_dev[dev];
  cudaStream_t st = (cudaStream_t)stream;

  // a throw-away host-side state that points the regular launchers at the caller's buffers and
  // at the fixed scratch: one worker pair each (n = 2), pair index 0
  cdgrab_ctx c;
  memset(&c, 0, sizeof(c));
  c.magic = CDG_MAGIC;
  c.m = m; c.n = 2; c.d = d; c.dtype = dtype;
  c.device = dev; c.num_sms = nd.num_sms;
  c.path = CDGRAB_PATH_FMA; c.k = 0; c.epoch_open = 1;
  c.r = r_dev;
  c.signs = signs_out_dev;
  c.partials = reinterpret_cast<double *>(nd.scratch + kOffPartials);
  c.gram = reinterpret_cast<double *>(nd.scratch + kOffGram);
  c.rnorm2 = reinterpret_cast<double *>(nd.scratch + kOffRnorm2);
  c.status = reinterpret_cast<int *>(nd.scratch + kOffStatus);
  c.perm_cur = reinterpret_cast<int32_t *>(nd.scratch + kOffPermCur);
  c.perm_next = reinterpret_cast<int32_t *>(nd.scratch + kOffPermNext);
  c.margins = reinterpret_cast<float *>(nd.scratch + kOffMargins);
  long long blocks = (d / 4 + 255) / 256;
  const long long cap = (long long)nd.num_sms * 2 < kNaMaxBlocks ? (long long)nd.num_sms * 2 : kNaMaxBlocks;
  if (blocks > cap) blocks = cap;
  c.gram_chunks = (int)blocks;

  // the tracked squared norm is read before it is written; the status word beside it is sticky
  // (bits only ever get set by the kernels) until cdgrab_noalloc_status reads and clears it
  if (cudaMemsetAsync(nd.scratch + kOffRnorm2, 0, 8, st) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  cudaError_t e = cdg_launch_gram_fma(&c, grads_dev, st);
  if (e == cudaSuccess) e = cdg_launch_scan(&c, st);
  if (e == cudaSuccess) e = cdg_launch_update(&c, grads_dev, st);
  if (e != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  return CDGRAB_OK;
}

// What the kernels of cdgrab_step_noalloc reported on the current device since the last call of
// this function: the status word sits in the fixed scratch, where no caller could read it.
// Synchronises the device, copies the word out, clears it when it is set.  Allocates nothing.
extern "C" int cdgrab_noalloc_status(void) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_DEVICE; }
  if (dev < 0 || dev >= kNaMaxDevices) return CDGRAB_ERR_DEVICE;
  const NaDevice &nd = g_na_dev[dev];
  if (!nd.ready) return CDGRAB_OK;             // no step has run on this device yet
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return CDGRAB_ERR_CUDA; }
  int st = 0;
  if (cudaMemcpy(&st, nd.scratch + kOffStatus, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return CDGRAB_ERR_CUDA;
  }
  if (st != 0) {
    const int zero = 0;
    if (cudaMemcpy(nd.scratch + kOffStatus, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaGetLastError();
      return CDGRAB_ERR_CUDA;
    }
  }
  if (st & CDG_ST_TIMEOUT) return CDGRAB_ERR_TIMEOUT;
  if (st & CDG_ST_NONFINITE) return CDGRAB_ERR_NONFINITE;
  return CDGRAB_OK;
}
