// dsvt_partition_noalloc: the rotated set partition for callers that must not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- inside a real-time perception loop
// whose memory budget is fixed at start-up, under a framework whose allocator owns the whole device,
// or in a plug-in that is handed a stream and buffers and nothing else.  dsvt_create reserves its
// workspace with cudaMalloc, so such callers cannot use a dsvt_ctx at all.  Here the sort buffers, the
// digit histograms and the per-window arrays live in one fixed array that is part of the library
// image; every GPU that loads the library holds it (about 1.9 MB) until the process exits.
#include <mutex>

#include "dsvt_common.cuh"

namespace {

constexpr int64_t kMaxVoxels = DSVT_NOALLOC_MAX_VOXELS;
constexpr int64_t kMaxWindows = DSVT_NOALLOC_MAX_WINDOWS;
constexpr int kMaxDevices = 64;

constexpr size_t pad256(size_t bytes) { return (bytes + 255) / 256 * 256; }
constexpr size_t kSortTiles = (size_t)(kMaxVoxels + 2047) / 2048 + 1;
constexpr size_t kOffStatus = 0;
constexpr size_t kOffKeys0 = kOffStatus + pad256(64 * 4);
constexpr size_t kOffKeys1 = kOffKeys0 + pad256((size_t)kMaxVoxels * 4);
constexpr size_t kOffVals0 = kOffKeys1 + pad256((size_t)kMaxVoxels * 4);
constexpr size_t kOffVals1 = kOffVals0 + pad256((size_t)kMaxVoxels * 4);
constexpr size_t kOffHist = kOffVals1 + pad256((size_t)kMaxVoxels * 4);
constexpr size_t kOffScanTmp = kOffHist + pad256((256 * kSortTiles + 1) * 4);
constexpr size_t kOffWinCount = kOffScanTmp + pad256(64 * 4);
constexpr size_t kOffWinStart = kOffWinCount + pad256((size_t)(kMaxWindows + 1) * 4);
constexpr size_t kOffWinSetoff = kOffWinStart + pad256((size_t)(kMaxWindows + 1) * 4);
constexpr size_t kScratchBytes = kOffWinSetoff + pad256((size_t)(kMaxWindows + 1) * 4);

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a
// device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {};  // device address of the array, per device

// Looks up (once per device, with that device current) where the array lives on the current device.
int scratch_for_current_device(unsigned char** out, int* cuda_err) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { *cuda_err = (int)e; return DSVT_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return DSVT_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) { *cuda_err = (int)e; return DSVT_ERR_CUDA; }
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return DSVT_OK;
}

}  // namespace

extern "C" int dsvt_partition_noalloc(void* cuda_stream, const int32_t* coords, int32_t n, int32_t batch,
                                      const int32_t grid[3], const int32_t window[3], int32_t set_size, int32_t axis,
                                      int32_t* set_table, int32_t cap_sets, int32_t* num_sets, int32_t* set_rowoff,
                                      int32_t* status_bits, int32_t* cuda_error) {
  int cuda_err = 0;
  if (cuda_error) *cuda_error = 0;
  if (!grid || !window) return DSVT_ERR_INVALID_ARG;
  if (n > kMaxVoxels) return DSVT_ERR_CAPACITY;  // more voxels than the fixed scratch can sort
  for (int a = 0; a < 3; ++a)
    if (grid[a] < 1 || window[a] < 1) return DSVT_ERR_INVALID_ARG;
  if (batch < 1) return DSVT_ERR_INVALID_ARG;
  int64_t windows = batch;
  for (int a = 0; a < 3; ++a) {
    windows *= dsvt_ceil_div(grid[a], window[a]);
    if (windows > kMaxWindows) return DSVT_ERR_CAPACITY;  // more windows than the fixed scratch holds
  }
  unsigned char* base = nullptr;
  int rc = scratch_for_current_device(&base, &cuda_err);
  if (rc != DSVT_OK) {
    if (cuda_error) *cuda_error = cuda_err;
    return rc;
  }
  // A context on the host stack whose workspace pointers all point into the fixed array: the partition
  // kernels run exactly as they do for a dsvt_create'd context, and nothing is allocated or freed.
  dsvt_ctx c = {};
  cudaGetDevice(&c.device);
  c.stream = (cudaStream_t)cuda_stream;
  c.max_voxels = kMaxVoxels;
  c.max_windows = kMaxWindows;
  c.max_channels = 0;
  c.status = reinterpret_cast<int32_t*>(base + kOffStatus);
  c.keys[0] = reinterpret_cast<uint32_t*>(base + kOffKeys0);
  c.keys[1] = reinterpret_cast<uint32_t*>(base + kOffKeys1);
  c.vals[0] = reinterpret_cast<int32_t*>(base + kOffVals0);
  c.vals[1] = reinterpret_cast<int32_t*>(base + kOffVals1);
  c.hist = reinterpret_cast<int32_t*>(base + kOffHist);
  c.scan_tmp = reinterpret_cast<int32_t*>(base + kOffScanTmp);
  c.win_count = reinterpret_cast<int32_t*>(base + kOffWinCount);
  c.win_start = reinterpret_cast<int32_t*>(base + kOffWinStart);
  c.win_setoff = reinterpret_cast<int32_t*>(base + kOffWinSetoff);
  // The array keeps whatever the previous call left: the status word must start at zero (the window
  // counters are cleared by the partition itself; everything else is written before it is read).
  cudaError_t e = cudaMemsetAsync(c.status, 0, sizeof(int32_t), c.stream);
  if (e != cudaSuccess) {
    if (cuda_error) *cuda_error = (int)e;
    return DSVT_ERR_CUDA;
  }
  rc = dsvt_partition(&c, coords, n, batch, grid, window, set_size, axis, set_table, cap_sets, num_sets, set_rowoff,
                      nullptr, nullptr, nullptr, nullptr);
  if (rc == DSVT_OK && status_bits) {
    e = cudaMemcpyAsync(status_bits, c.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, c.stream);
    if (e != cudaSuccess) { c.last_cuda_error = (int)e; rc = DSVT_ERR_CUDA; }
  }
  if (cuda_error) *cuda_error = c.last_cuda_error;
  return rc;
}
