// qadam_worker_scales_static: the max-abs scales of the worker side without any
// allocation, for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all once they are running:
// a process that sizes all of its device memory at start-up and forbids later
// allocation (hard real-time loops, memory-capped multi-tenant services), or code
// that runs where an allocation would synchronise the device in the middle of its
// work.  The regular entry points never allocate either, but they need a
// caller-provided workspace, which such a caller would itself have had to
// allocate.  This entry point needs none: its scratch (the tile table the kernel
// walks and the per-worker accumulators of the running maximum) lives in a
// fixed-size array that is part of the library image on every GPU that loads it.
#include "qadam.h"

#include <cuda_runtime.h>

#include <mutex>

#include "qadam_host.h"
#include "qadam_kernels.cuh"

using namespace qadam;

namespace {

constexpr int kStaticMaxWorkers = QADAM_STATIC_MAX_WORKERS;
constexpr long long kStaticMaxElems = QADAM_STATIC_MAX_ELEMENTS;
constexpr int kStaticMaxTiles = (int)(kStaticMaxElems / kTileElems);      // 16384
constexpr size_t kAccBytes = sizeof(unsigned) * kStaticMaxWorkers;          // 4 KiB
constexpr size_t kScratchBytes = kAccBytes + sizeof(Tile) * (size_t)kStaticMaxTiles;   // 260 KiB

// The scratch.  Every GPU that loads the library holds these 260 KiB until the
// process exits.  Layout: [per-worker accumulators][tile table].
// In host code this name is only a handle for cudaGetSymbolAddress, never an address.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
  void* scratch = nullptr;   // device address of the array on this device
  int grid = 0;              // CTAs that keep the device full with the max-abs kernel
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

inline bool cuda_ok(cudaError_t e) {
  if (e != cudaSuccess) {
    record_cuda_error((int)e);
    return false;
  }
  return true;
}

// Address of the scratch and launch width on the current device; looked up once per
// device, before anything is enqueued.
int setup_for_current_device(DeviceSetup* out) {
  int dev = 0;
  if (!cuda_ok(cudaGetDevice(&dev))) return QADAM_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return QADAM_ERR_CAPACITY;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& d = g_setup[dev];
  if (d.scratch == nullptr) {
    void* ptr = nullptr;
    int sms = 0, per_sm = 0;
    if (!cuda_ok(cudaGetSymbolAddress((void**)&ptr, g_static_scratch)) || ptr == nullptr ||
        !cuda_ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) ||
        !cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, worker_absmax_kernel<false>, kThreads, 0)))
      return QADAM_ERR_CUDA;
    d.grid = sms * (per_sm > 0 ? per_sm : 1);
    d.scratch = ptr;
  }
  *out = d;
  return QADAM_OK;
}

// Writes the tile table of one flat segment of D elements into the scratch.
__global__ void static_fill_tiles_kernel(Tile* tiles, long long D, int num_tiles) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= num_tiles) return;
  const long long off = (long long)t * kTileElems;
  const long long left = D - off;
  Tile tile;
  tile.off = off;
  tile.count = (int)(left < kTileElems ? left : kTileElems);
  tile.seg = 0;
  tiles[t] = tile;
}

__global__ void static_copy_scales_kernel(const unsigned* acc, float* scales, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) scales[i] = __uint_as_float(acc[i]);
}

}  // namespace

extern "C" int qadam_worker_scales_static(const float* g, const float* e, int64_t D, int32_t n,
                                          float* scales, void* stream) {
  if (!g || !e || !scales) return QADAM_ERR_NULL;
  if (D < 1 || n < 1 || D % kAlign != 0) return QADAM_ERR_SIZE;
  if (D > kStaticMaxElems || n > kStaticMaxWorkers) return QADAM_ERR_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(e)) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(scales) % 4 != 0)
    return QADAM_ERR_ALIGN;
  DeviceSetup setup;
  const int rc = setup_for_current_device(&setup);
  if (rc != QADAM_OK) return rc;
  void* scratch = setup.scratch;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned* acc = static_cast<unsigned*>(scratch);
  Tile* tiles = reinterpret_cast<Tile*>(static_cast<unsigned char*>(scratch) + kAccBytes);
  const int num_tiles = (int)((D + kTileElems - 1) / kTileElems);

  // The array still holds the previous call's table and maxima: rewrite the table for
  // this D and clear the accumulators, which must start at zero.
  if (!cuda_ok(cudaMemsetAsync(acc, 0, sizeof(unsigned) * (size_t)n, st))) return QADAM_ERR_CUDA;
  static_fill_tiles_kernel<<<(num_tiles + 255) / 256, 256, 0, st>>>(tiles, (long long)D, num_tiles);
  if (!cuda_ok(cudaGetLastError())) return QADAM_ERR_CUDA;

  WorkerParams p;
  p.g = g;
  p.m = nullptr; p.v = nullptr;
  p.e = const_cast<float*>(e);          // phase 1 with the moments on the server only reads e
  p.scale_bits = acc;
  p.gcodes = nullptr;
  p.tiles = tiles;
  p.status = nullptr;
  p.D = D;
  p.gcode_bytes = 0;
  p.tiles_per_worker = num_tiles;
  p.total_tiles = (long long)n * num_tiles;
  p.S = 1;
  p.worker_begin = 0;
  p.k = 0; p.L = 1; p.bits = 2;
  p.alpha = 0.0f;
  p.h = Hyper{0.0f, 0.0f, 1.0f, 1.0f, 1.0f};
  p.x = nullptr; p.wcodes = nullptr; p.kx = -1; p.xbits = 0; p.lambda = 0.0f;   // no l2 term
  p.spin_limit = 0;
  p.seed_lo = p.seed_hi = p.step = 0;

  long long grid = setup.grid;
  if (grid > p.total_tiles) grid = p.total_tiles;
  worker_absmax_kernel<false><<<(int)grid, kThreads, 0, st>>>(p);
  if (!cuda_ok(cudaGetLastError())) return QADAM_ERR_CUDA;
  static_copy_scales_kernel<<<(n + 255) / 256, 256, 0, st>>>(acc, scales, n);
  if (!cuda_ok(cudaGetLastError())) return QADAM_ERR_CUDA;
  return QADAM_OK;
}
