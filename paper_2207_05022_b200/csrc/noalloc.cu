// Allocation-free decode of one shard matrix.
//
// sti_shard_decode works on a plan, and a plan keeps its re-tiled index streams, tables and outlier
// lists in arenas it obtained from cudaMalloc / cudaMallocHost.  Some callers must not allocate:
// a loader that verifies a shard file inside a serving process whose framework allocator already owns
// the device memory, a health check that runs while a memory budget is enforced, code that runs in a
// section where the CUDA allocator's implicit synchronisation is not acceptable.  For them this file
// offers the same decode kernel with its working copy of the shard in a fixed device array that is
// part of the library image: every GPU on which the library is loaded carries these
// STI_NOALLOC_SCRATCH_BYTES (about 288 KiB) until the process exits.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/sti.h"
#include "retile.h"
#include "sti_kernels.h"

namespace {

constexpr size_t kCodesMax = 262144;          // bytes of one matrix's index stream (rows * cols * bits / 8)
constexpr size_t kTableBytes = 256;           // 64 fp32 centroids
constexpr size_t kOutliersMax = 4096;         // outliers of one matrix
constexpr size_t kOffCodes = 0;
constexpr size_t kOffTable = kCodesMax;
constexpr size_t kOffOutOff = kOffTable + kTableBytes;
constexpr size_t kOffOutVal = kOffOutOff + kOutliersMax * 4;
constexpr size_t kScratchBytes = kOffOutVal + kOutliersMax * 4;
static_assert(kScratchBytes == STI_NOALLOC_SCRATCH_BYTES, "header and implementation disagree on the scratch size");

// The scratch itself.  In host code this name is only a handle for the runtime's symbol calls,
// never a device address; the address is looked up once per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;                           // one call at a time: the host staging buffer is shared too
unsigned char* g_scratch_dev[kMaxDevices] = {};
bool g_ready[kMaxDevices] = {};
// Host side of the staging, shared by all calls (hence the mutex): pageable on purpose, so that cudaMemcpyAsync
// has read it by the time it returns and the next call may overwrite it.
unsigned char g_host_stage[kCodesMax];        // re-tiled stream on its way to the device
float g_host_table[64];
uint32_t g_host_off[kOutliersMax];
float g_host_val[kOutliersMax];

// Puts the caller's current device back when the call returns, whatever the outcome.
struct DeviceGuard {
  int prev = -1;
  DeviceGuard() { if (cudaGetDevice(&prev) != cudaSuccess) { (void)cudaGetLastError(); prev = -1; } }
  ~DeviceGuard() { if (prev >= 0) (void)cudaSetDevice(prev); }
};

}  // namespace

extern "C" sti_status sti_matrix_decode_noalloc(int device, void* stream, int bits, uint32_t rows, uint32_t cols,
                                                const uint32_t* codes, const float* centroids,
                                                const uint32_t* outlier_off, const float* outlier_val,
                                                size_t n_outliers, float* w_dev, uint8_t* codes_dev,
                                                uint16_t* wbf16_dev) {
  // ---- argument checks first: nothing below is reached with a size the scratch cannot hold
  if (!codes || !centroids) return STI_ERR_ARG;
  if (!w_dev && !codes_dev && !wbf16_dev) return STI_ERR_ARG;
  if (device < 0 || device >= kMaxDevices) return STI_ERR_ARG;
  if (bits < 2 || bits > 6) return STI_ERR_BITS;
  if (rows == 0 || cols == 0) return STI_ERR_SHAPE;
  if (cols == 64 ? rows % 64 != 0 : (cols % 128 != 0 || rows % 32 != 0)) return STI_ERR_SHAPE;
  const unsigned long long n = static_cast<unsigned long long>(rows) * cols;
  const unsigned long long stream_bytes = n * static_cast<unsigned>(bits) / 8;
  if (stream_bytes > kCodesMax) return STI_ERR_SIZE;            // matrix larger than the fixed scratch
  if (n_outliers > kOutliersMax) return STI_ERR_SIZE;           // more outliers than the fixed scratch holds
  if (n_outliers && (!outlier_off || !outlier_val)) return STI_ERR_ARG;
  for (size_t i = 0; i < n_outliers; ++i) {
    if (outlier_off[i] >= n) return STI_ERR_SIZE;
    if (i && outlier_off[i] <= outlier_off[i - 1]) return STI_ERR_ARG;
  }

  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceGuard restore_device;
  if (cudaSetDevice(device) != cudaSuccess) {
    (void)cudaGetLastError();
    return STI_ERR_CUDA;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The copies below read host buffers that the next call reuses and that the caller may free: inside a stream
  // capture they would only be read when the graph runs.  Such a call is refused.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) {
    (void)cudaGetLastError();
    return STI_ERR_CUDA;
  }
  if (cap != cudaStreamCaptureStatusNone) return STI_ERR_STATE;
  // ---- first call on this device: find out where the device array lives (not an allocation)
  if (!g_ready[device]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return STI_ERR_CUDA;
    }
    g_scratch_dev[device] = static_cast<unsigned char*>(p);
    g_ready[device] = true;
  }
  unsigned char* scratch = g_scratch_dev[device];

  // ---- stage the shard into the scratch: the array still holds the previous call's shard, so every
  // region the kernel will read is overwritten here (stream, table, outlier lists); nothing else is read
  sti::retile_matrix(reinterpret_cast<const unsigned char*>(codes), g_host_stage, rows, cols,
                     static_cast<uint32_t>(bits));
  for (int i = 0; i < 64; ++i) g_host_table[i] = i < (1 << bits) ? centroids[i] : 0.f;
  // the outlier lists go through library-owned pageable buffers too: the caller's arrays may be pinned, and a copy
  // out of pinned memory would still be reading them after this call has returned
  for (size_t i = 0; i < n_outliers; ++i) { g_host_off[i] = outlier_off[i]; g_host_val[i] = outlier_val[i]; }
  auto fail = [] { (void)cudaGetLastError(); return STI_ERR_CUDA; };      // leave no sticky error behind
  if (cudaMemcpyAsync(scratch + kOffCodes, g_host_stage, stream_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(scratch + kOffTable, g_host_table, kTableBytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return fail();
  if (n_outliers) {
    if (cudaMemcpyAsync(scratch + kOffOutOff, g_host_off, n_outliers * 4, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(scratch + kOffOutVal, g_host_val, n_outliers * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
      return fail();
  }
  sti::DecodeLaunch dl{};
  dl.codes = reinterpret_cast<const uint4*>(scratch + kOffCodes);
  dl.table = reinterpret_cast<const float*>(scratch + kOffTable);
  dl.out_off = reinterpret_cast<const uint32_t*>(scratch + kOffOutOff);
  dl.out_val = reinterpret_cast<const float*>(scratch + kOffOutVal);
  dl.n_out = static_cast<uint32_t>(n_outliers);
  dl.flat_base = 0;
  dl.bits = static_cast<uint32_t>(bits);
  dl.rows = rows;
  dl.kc = cols;
  dl.w = w_dev;
  dl.codes_out = codes_dev;
  dl.wbf16 = wbf16_dev;
  if (sti::launch_decode(dl, s) != cudaSuccess) return fail();
  return STI_OK;
}
