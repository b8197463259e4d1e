// Device-side descriptors and launchers of the gather / scatter movers.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace kvr {

// One request's share of one launch.  Tiles of a request are numbered
// q = plane * nb + b (plane = 2*layer + kv, b = logical block), which is also
// the order of their bytes in the image, so a run of tile ids is one
// contiguous byte range of the image.
struct Seg {
  const int32_t *bt;     // DEVICE: the request's block table (nb entries)
  char *img;             // address of image byte 0 in the linear buffer this launch reads or writes
                         // (may lie before the buffer when the launch covers a later part of the image)
  long long n_tokens;
  long long tile_begin;  // first tile id of this request handled by the launch
  long long tile_count;
  int nb;
  int pad;
};

constexpr int kMaxSegs = 1024;   // segments per launch (the host splits larger batches)

struct MoveArgs {
  const Seg *segs;       // DEVICE
  int nsegs;
  long long total_tiles; // sum of tile_count
  char *pool;            // DEVICE: paged pool base
  long long plane_stride;// bytes from one (layer, plane) to the next, for a fixed block
  long long block_stride;// bytes from one block to the next, for a fixed plane
  int tile_bytes;        // block_size * row_bytes
  int row_bytes;         // kv_heads * head_dim * dtype_bytes (multiple of 16)
  int block_size;
  int num_blocks;        // blocks in the pool: a table entry outside [0, num_blocks) is never dereferenced (0 = unchecked)
  int *status;           // DEVICE or NULL: error word (0 = fine); 1 = a bounded wait ran out, 3 = a table entry out of range
  unsigned long long *stamp;  // DEVICE or NULL: stamp[0] = earliest start, stamp[1] = latest end of any CTA, in
                              // %globaltimer nanoseconds (the host initialises them to ~0 and 0)
  unsigned long long *work;   // DEVICE: work counter of this launch, zero when the kernel starts.  The movers hand out
                              // work through it (whoever is free takes the next unit), so all SMs finish together.
};

struct BulkShape {       // tuning of the bulk mover
  int warps;             // independent pipelines per CTA
  int stages;            // shared-memory stages per pipeline
  int piece_bytes;       // bytes per bulk copy (multiple of 16, <= tile_bytes rounded)
};

// gather = pool -> linear, scatter = linear -> pool.  grid_limit caps the number of CTAs (0 = default).
cudaError_t launch_move_warp(bool gather, const MoveArgs &a, int grid_limit, int sm_count, cudaStream_t s);
cudaError_t launch_move_bulk(bool gather, const MoveArgs &a, const BulkShape &shape, int grid_limit,
                             int sm_count, cudaStream_t s);
cudaError_t bulk_configure(const BulkShape &shape);   // once per device: opt in to large dynamic shared memory

// `launches` back-to-back streaming reads of buf (benchmark load); sink = 8 KiB of device memory
cudaError_t launch_read_load(const void *buf, unsigned long long bytes, int launches, void *sink, cudaStream_t s);

// one thread waits `limit` polls on an mbarrier nobody completes, then writes 2 to *status (pinned host word)
cudaError_t launch_wait_limit_probe(int *status, unsigned limit, cudaStream_t s);

constexpr int kStatusWaitRanOut = 1, kStatusProbe = 2, kStatusBadBlock = 3;

}  // namespace kvr
