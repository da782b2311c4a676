// sortLSH of one matrix without any allocation.
//
// Some callers of this library are not allowed to allocate device memory once they are
// running: an inference server that carves up HBM at start-up and forbids cudaMalloc
// afterwards, a plug-in loaded into a process whose allocator is owned by someone else, a
// real-time loop that may not take the driver's allocation locks.  For them this file offers
// one entry point whose scratch memory is a fixed array that is part of the library image.
// The price: every GPU that loads the library holds the array (kScratchBytes) until the
// process exits, the problem size is capped, and all calls share the one array.
#include <mutex>

#include "../../include/hyperattn.h"
#include "common.cuh"

namespace hyperattn {
namespace {

constexpr int kNoAllocMaxRows = HYPERATTN_NOALLOC_MAX_ROWS;
constexpr size_t kChunksMax = (kNoAllocMaxRows + kSortChunk - 1) / kSortChunk;
// layout of the scratch array (bytes): ids | chunk histograms | chunk offsets (the matrix is the "key" side of
// a one-segment problem that has no query rows)
constexpr size_t kOffIds = 0;
constexpr size_t kOffHist = kOffIds + (size_t)kNoAllocMaxRows;
constexpr size_t kOffOffs = kOffHist + kChunksMax * kBuckets * 4;
constexpr size_t kScratchBytes = kOffOffs + kChunksMax * kBuckets * 4;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices];     // device ordinal -> device address of g_scratch (a fixed table: no heap)

// First call on a device: resolve the array's device address (with that device current).
int scratch_for_current_device(unsigned char** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  if (dev < 0 || dev >= kMaxDevices) return HYPERATTN_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return HYPERATTN_CUDA_ERROR;
    }
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return HYPERATTN_OK;
}

}  // namespace
}  // namespace hyperattn

using namespace hyperattn;

extern "C" int hyperattn_sortlsh_noalloc(const void* x, int n, int d, int hash_bits, uint64_t seed,
                                         uint8_t* ids, int32_t* perm, int32_t* rank, void* stream) {
  if (!x || !ids || !perm || !rank) return HYPERATTN_INVALID_ARGUMENT;
  if (n <= 0) return HYPERATTN_INVALID_ARGUMENT;
  if (d != 64 && d != 128) return HYPERATTN_UNSUPPORTED_SHAPE;
  if (hash_bits < 1 || hash_bits > 8) return HYPERATTN_UNSUPPORTED_SHAPE;
  if (n > kNoAllocMaxRows) return HYPERATTN_UNSUPPORTED_SHAPE;   // beyond the built-in scratch: use hyperattn_forward_ex
  if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(perm) & 3) || (reinterpret_cast<uintptr_t>(rank) & 3))
    return HYPERATTN_MISALIGNED;
  unsigned char* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc) return rc;

  // One segment whose key side is the matrix and whose query side has no rows and no chunks: the key side
  // carries the inverse permutation that callers want, and nothing of the other side is read, hashed or placed.
  Geometry g = {};
  g.G = 1; g.n = 0; g.nk = n; g.npad = 0; g.d = d; g.b = 1; g.bq = 1; g.m = 0; g.r = hash_bits;
  g.causal = 0; g.L = 0; g.leaf = 0; g.unit = 1; g.unit_k = n;
  g.chunks_per_unit = 0; g.chunks_per_seg = 0;
  g.chunks_per_unit_k = (n + kSortChunk - 1) / kSortChunk;
  g.chunks_per_seg_k = g.chunks_per_unit_k;
  g.levels = 1; g.nl = n; g.nodes = 1; g.sorted = 1;

  Workspace ws = {};
  ws.ids = scratch + kOffIds;                                          // [n]: fully rewritten by the hash kernel
  ws.hist = reinterpret_cast<uint32_t*>(scratch + kOffHist);          // fully rewritten by the hash kernel
  ws.offs = reinterpret_cast<uint32_t*>(scratch + kOffOffs);          // fully rewritten by the scan kernel
  ws.perm_k = perm;
  ws.rank_k = rank;

  float w[128 * 8];
  hyperattn_get_projections(d, hash_bits, seed, w);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  constexpr int kKeysOnly = 2;
  if (launch_hash(g, nullptr, x, /*is_fp32=*/0, w, ws, nullptr, st, kKeysOnly) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  if (launch_sort_scan(g, ws, false, 0, st, kKeysOnly) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  if (launch_sort_scatter(g, ws, st, kKeysOnly) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  if (cudaMemcpyAsync(ids, ws.ids, (size_t)n, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return HYPERATTN_CUDA_ERROR;
  return HYPERATTN_OK;
}
