// kvr_gather_noalloc: the gather kernel for callers that cannot allocate.
//
// Who that is: a serving engine that has handed every byte of device memory to its own KV-block
// allocator (so a cudaMalloc inside a helper would fail, or would shrink the pool it sized to fill the
// GPU), and code on a latency-critical path where the device-wide synchronisation that cudaMalloc and
// cudaFree imply is not acceptable.  For them the descriptors the gather kernel reads -- one segment
// record and the request's block table -- live in a fixed array in the library's device image instead
// of a buffer allocated per pool.  The caller still owns and passes the pool and the destination.
//
// Cost and limits: every GPU that loads this library carries the array (about 256 KiB) until the
// process exits; one call moves one request of at most KVR_NOALLOC_MAX_BLOCKS blocks; all calls share
// the array, so two calls whose GPU work can overlap (different streams, or different host threads)
// race on it -- issue them on one stream, or wait for the first before starting the second.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/kvr.h"
#include "kvr_kernels.cuh"

namespace kvr { void set_last_error(const char *msg); }

namespace {

constexpr size_t kSegBytes = 256;   // the segment record, padded so the table that follows stays 256-byte aligned
constexpr size_t kWorkOffset = 128; // inside that padding: the launch's work counter, uploaded as zero with the record
static_assert(sizeof(kvr::Seg) <= kWorkOffset, "the work counter would overlap the segment record");
constexpr size_t kScratchBytes = kSegBytes + sizeof(int32_t) * (size_t)KVR_NOALLOC_MAX_BLOCKS;

// Scratch of the allocation-free entry point.  In host code this name is only a handle for
// cudaGetSymbolAddress(): it is not a device address and must never be passed to a kernel as is.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// Host-side twin of the array: the record and the table are first copied here, checked here, and uploaded from
// here.  It is ordinary pageable memory, so the runtime has taken its own copy of it by the time each
// cudaMemcpyAsync returns; the caller's table (pageable or page-locked) is read only during the call, and the ids
// the kernel sees are exactly the ids that were range-checked.  g_stage_mu serialises the host side of calls.
alignas(256) unsigned char g_stage[kScratchBytes];
std::mutex g_stage_mu;

constexpr int kMaxDevices = 64;
unsigned char *g_scratch_ptr[kMaxDevices];   // device address of the array, per device ordinal (set up on first use)
int g_sm_count[kMaxDevices];

kvr_status fail_na(kvr_status st, const char *msg) { kvr::set_last_error(msg); return st; }

// Once per device, with that device current: resolve the array's device address.
kvr_status setup_device(int dev) {
  if (g_scratch_ptr[dev]) return KVR_OK;
  void *ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
  if (e != cudaSuccess || !ptr) {
    char buf[256];
    snprintf(buf, sizeof buf, "cudaGetSymbolAddress(scratch) failed on device %d: %s", dev, cudaGetErrorString(e));
    return fail_na(KVR_ERR_CUDA, buf);
  }
  int sms = 0;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess || sms < 1) return fail_na(KVR_ERR_CUDA, "cudaDeviceGetAttribute(multiprocessor count) failed");
  g_sm_count[dev] = sms;
  g_scratch_ptr[dev] = static_cast<unsigned char *>(ptr);
  return KVR_OK;
}

}  // namespace

extern "C" kvr_status kvr_gather_noalloc(const void *device_pool, const kvr_geometry *g, int32_t num_blocks,
                                         const int32_t *block_table, int32_t nb, int64_t n_tokens,
                                         void *dst_device, void *stream) {
  const uint64_t bpt = kvr_bytes_per_token(g);
  if (!bpt) return fail_na(KVR_ERR_GEOMETRY, "invalid geometry");
  if (!device_pool || !dst_device || num_blocks < 1 || n_tokens < 0 || nb < 0 || (nb > 0 && !block_table))
    return fail_na(KVR_ERR_INVALID_ARG, "NULL pointer or negative size");
  if (((uintptr_t)device_pool & 15) || ((uintptr_t)dst_device & 15))
    return fail_na(KVR_ERR_INVALID_ARG, "device_pool and dst_device must be 16-byte aligned");
  if (nb > KVR_NOALLOC_MAX_BLOCKS) {
    char buf[256];
    snprintf(buf, sizeof buf, "request has %d blocks; kvr_gather_noalloc holds at most %d (KVR_NOALLOC_MAX_BLOCKS) "
             "in its fixed scratch: split the request or use kvr_export_to_device", nb, KVR_NOALLOC_MAX_BLOCKS);
    return fail_na(KVR_ERR_INVALID_ARG, buf);
  }
  if ((n_tokens + g->block_size - 1) / g->block_size != nb)
    return fail_na(KVR_ERR_INVALID_ARG, "nb must equal ceil(n_tokens / block_size)");
  // sizes in 64 bits: a tile is at most 1 GiB (the same rule as kvr_pool_create), so the kernel's int fields hold
  const uint64_t row = bpt / 2 / (uint64_t)g->layers;
  const uint64_t tile = row * (uint64_t)g->block_size;
  if (tile > (1ull << 30)) return fail_na(KVR_ERR_GEOMETRY, "one tile exceeds 1 GiB");
  if (nb == 0) return KVR_OK;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fail_na(KVR_ERR_CUDA, "no current CUDA device (or ordinal >= 64)");
  if (kvr_status s = setup_device(dev)) return s;
  unsigned char *scratch = g_scratch_ptr[dev];
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  kvr::Seg seg{};
  seg.bt = reinterpret_cast<const int32_t *>(scratch + kSegBytes);
  seg.img = static_cast<char *>(dst_device);
  seg.n_tokens = n_tokens;
  seg.tile_begin = 0;
  seg.tile_count = 2ll * g->layers * nb;
  seg.nb = nb;

  {
    std::lock_guard<std::mutex> hold(g_stage_mu);
    int32_t *table = reinterpret_cast<int32_t *>(g_stage + kSegBytes);
    memcpy(g_stage, &seg, sizeof seg);
    memset(g_stage + kWorkOffset, 0, sizeof(unsigned long long));
    memcpy(table, block_table, sizeof(int32_t) * (size_t)nb);
    for (int32_t i = 0; i < nb; ++i)
      if (table[i] < 0 || table[i] >= num_blocks) return fail_na(KVR_ERR_INVALID_ARG, "block id out of range");
    // One upload of record + table from the pageable twin: the runtime copies a pageable source out before the call
    // returns (after waiting for whatever `stream` ran before), so the twin is free again when the lock drops.  The
    // upload is ordered on `stream` before the kernel and after the previous call's kernel.
    cudaError_t e = cudaMemcpyAsync(scratch, g_stage, kSegBytes + sizeof(int32_t) * (size_t)nb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail_na(KVR_ERR_CUDA, cudaGetErrorString(e));
  }

  kvr::MoveArgs a{};
  a.segs = reinterpret_cast<const kvr::Seg *>(scratch);
  a.nsegs = 1;
  a.total_tiles = seg.tile_count;
  a.pool = static_cast<char *>(const_cast<void *>(device_pool));
  a.tile_bytes = (int)tile;
  a.plane_stride = (long long)num_blocks * (long long)tile;   // layer-major pool
  a.block_stride = (long long)tile;
  a.row_bytes = (int)row;
  a.block_size = g->block_size;
  a.num_blocks = num_blocks;
  a.status = nullptr;               // the warp mover has no bounded waits, and the table was checked above
  a.work = reinterpret_cast<unsigned long long *>(scratch + kWorkOffset);
  cudaError_t e = kvr::launch_move_warp(true, a, 0, g_sm_count[dev], st);
  if (e != cudaSuccess) return fail_na(KVR_ERR_CUDA, cudaGetErrorString(e));
  return KVR_OK;
}
