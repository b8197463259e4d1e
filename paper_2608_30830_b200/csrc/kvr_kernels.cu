// Gather / scatter movers for sm_100a.
//
// The work of one launch is a flat list of tiles.  A tile is the part of one
// block of one request that lies in one (layer, K|V) plane: up to
// block_size * row_bytes contiguous bytes in the pool and the same bytes,
// contiguous, in the linear image.  Requests are ragged (different block
// counts), so the flat tile id is mapped to (request, plane, block) through an
// exclusive prefix sum of the per-request tile counts, built once per CTA with
// warp shuffles and then searched per tile.
//
//   move_warp : one warp per tile, 16-byte loads and stores, 8 in flight per lane
//   move_bulk : one thread per pipeline drives bulk async copies
//               global -> shared -> global through a ring of shared-memory
//               stages guarded by mbarriers (every copy is issued and consumed by one
//               CTA: no tile is shared between CTAs)
//
// Work is handed out dynamically: a launch carries a zeroed counter and every
// pipeline (or warp) takes the next unit (32 KiB, or a few smaller ones) with
// one atomicAdd when it is free.
// SMs do not all reach HBM equally fast, so fixed equal shares leave most of
// the chip idle while the slowest SM finishes (measured: 6.2 TB/s with equal
// shares, 6.7-6.8 TB/s with the counter, on 2-4 GiB launches); claiming one
// unit at a time also keeps all pipelines inside one moving window of the
// image.
#include "kvr_kernels.cuh"

namespace kvr {

namespace {

constexpr int kWarpThreads = 256;          // threads per CTA of the warp mover
constexpr int kMaxBulkWarps = 8;
constexpr int kMaxBulkStages = 8;
constexpr unsigned kSpinLimit = 1u << 22;  // bounded mbarrier wait (each spin sleeps >= 32 ns after the first 64)
constexpr int kClaimBytes = 32 * 1024;     // work taken from a launch's counter per atomicAdd (at least one unit)

// Exclusive prefix sum of tile counts into cum[0..nsegs]; cum[nsegs] = total.
// Done by warp 0 in strides of 32 with shuffle-up, carrying the running total.
__device__ __forceinline__ void scan_segments(const MoveArgs &a, long long *cum) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    long long carry = 0;
    for (int base = 0; base < a.nsegs; base += 32) {
      const int i = base + lane;
      long long v = i < a.nsegs ? a.segs[i].tile_count : 0;
      long long incl = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        long long up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
      }
      if (i < a.nsegs) cum[i] = carry + incl - v;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) cum[a.nsegs] = carry;
  }
  __syncthreads();
}

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

struct Tile {
  char *pool_ptr;   // first byte of the tile in the pool
  char *lin_ptr;    // first byte of the tile in the linear image
  int bytes;        // valid bytes (a request's last block may be partial)
};

// flat tile id -> addresses.  cum is in shared memory; the search is uniform across a warp.
__device__ __forceinline__ Tile locate(const MoveArgs &a, const long long *cum, long long w) {
  int lo = 0, hi = a.nsegs - 1;
  while (lo < hi) {                       // last segment with cum[seg] <= w
    const int mid = (lo + hi + 1) >> 1;
    if (cum[mid] <= w) lo = mid; else hi = mid - 1;
  }
  const Seg sg = a.segs[lo];
  const long long q = sg.tile_begin + (w - cum[lo]);
  const long long plane = q / sg.nb;
  const int b = (int)(q - plane * sg.nb);
  const int blk = __ldg(sg.bt + b);
  const long long first_tok = (long long)b * a.block_size;
  long long valid = sg.n_tokens - first_tok;
  if (valid > a.block_size) valid = a.block_size;
  Tile t;
  // The host validates every table before it is uploaded; should an entry still arrive out of range, the tile is
  // skipped and the error word says so -- the pool is never addressed outside its extent.
  if (a.num_blocks > 0 && (unsigned)blk >= (unsigned)a.num_blocks) {
    if (a.status) { *reinterpret_cast<volatile int *>(a.status) = kStatusBadBlock; __threadfence_system(); }
    t.pool_ptr = a.pool; t.lin_ptr = sg.img; t.bytes = 0;
    return t;
  }
  t.pool_ptr = a.pool + plane * a.plane_stride + (long long)blk * a.block_stride;
  t.lin_ptr = sg.img + (plane * sg.n_tokens + first_tok) * a.row_bytes;
  t.bytes = (int)valid * a.row_bytes;
  return t;
}

// ---- warp mover --------------------------------------------------------------------

// One warp per tile; the warps of the grid take consecutive tiles from the launch's work counter, so at any moment
// the grid covers one contiguous window of the image.  A lane keeps 8
// independent 16-byte loads in flight (streaming cache policy: every byte is touched once) before it stores them.
template <bool GATHER>
__global__ void __launch_bounds__(kWarpThreads) move_warp_kernel(const MoveArgs a) {
  // (nsegs + 1) prefix sums, sized at launch (typically a few dozen bytes)
  extern __shared__ __align__(8) long long cum[];
  if (a.stamp && threadIdx.x == 0) atomicMin(a.stamp, global_ns());
  scan_segments(a, cum);
  const int lane = threadIdx.x & 31;
  // small tiles are claimed several at a time, so that the counter is not the bottleneck
  const int claim = a.tile_bytes >= kClaimBytes ? 1 : kClaimBytes / a.tile_bytes;
  long long next = 0, claim_end = 0;
  for (;;) {
    if (next >= claim_end) {
      unsigned long long first = 0;
      if (lane == 0) first = atomicAdd(a.work, (unsigned long long)claim);
      next = (long long)__shfl_sync(0xffffffffu, first, 0);
      claim_end = next + claim;
    }
    const long long w = next++;
    if (w >= a.total_tiles) break;
    const Tile t = locate(a, cum, w);
    const uint4 *src = reinterpret_cast<const uint4 *>(GATHER ? t.pool_ptr : t.lin_ptr);
    uint4 *dst = reinterpret_cast<uint4 *>(GATHER ? t.lin_ptr : t.pool_ptr);
    const int nvec = t.bytes >> 4;
    int i = lane;
    for (; i + 32 * 7 < nvec; i += 32 * 8) {
      uint4 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = __ldcs(src + i + 32 * k);
#pragma unroll
      for (int k = 0; k < 8; ++k) __stcs(dst + i + 32 * k, v[k]);
    }
    for (; i < nvec; i += 32) __stcs(dst + i, __ldcs(src + i));
  }
  if (a.stamp && lane == 0) atomicMax(a.stamp + 1, global_ns());     // every warp: the latest one wins
}

// ---- bulk mover ----------------------------------------------------------------------

__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit ran out (the caller records it and leaves).
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, unsigned limit = kSpinLimit) {
  for (unsigned spin = 0; spin < limit; ++spin) {
    if (mbar_test(bar, parity)) return true;
    if (spin > 64) __nanosleep(32);
  }
  return false;
}
__device__ __forceinline__ void bulk_load(unsigned dst_smem, const void *src, unsigned bytes, unsigned bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, unsigned src_smem, unsigned bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// STAGES shared-memory stages per pipeline; a store trails its load by LAG = STAGES/2 units,
// so LAG loads and STAGES-LAG stores are in flight per pipeline.  A pipeline takes its units from the launch's
// work counter, one at a time.
template <bool GATHER, int STAGES>
__global__ void __launch_bounds__(kMaxBulkWarps * 32) move_bulk_kernel(const MoveArgs a, const int piece_bytes) {
  constexpr int LAG = STAGES / 2 > 0 ? STAGES / 2 : 1;
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ long long cum[kMaxSegs + 1];
  __shared__ __align__(8) unsigned long long bars[kMaxBulkWarps][kMaxBulkStages];
  __shared__ char *pend_dst[kMaxBulkWarps][kMaxBulkStages];
  __shared__ int pend_len[kMaxBulkWarps][kMaxBulkStages];

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  if (a.stamp && threadIdx.x == 0) atomicMin(a.stamp, global_ns());
  if (lane == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(smem_addr(&bars[warp][s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  scan_segments(a, cum);   // ends with __syncthreads()
  if (lane != 0) return;

  const int pieces_per_tile = (a.tile_bytes + piece_bytes - 1) / piece_bytes;
  const long long total_units = a.total_tiles * pieces_per_tile;
  unsigned char *my_ring = ring + (size_t)warp * STAGES * piece_bytes;
  unsigned phase_bits = 0;
  bool failed = false, more = true;
  long long issued = 0, stored = 0;      // units whose load / store this pipeline has issued
  // small pieces are claimed several at a time, so that the counter is not the bottleneck
  const int claim = piece_bytes >= kClaimBytes ? 1 : kClaimBytes / piece_bytes;
  long long claim_next = 0, claim_end = 0;

  // Every turn issues the load of one more unit while there is one, and the store of the unit LAG behind it.
  for (;;) {
    if (more) {
      long long u;
      if (claim_next >= claim_end) {
        claim_next = (long long)atomicAdd(a.work, (unsigned long long)claim);
        claim_end = claim_next + claim;
      }
      u = claim_next++;
      if (u >= total_units) {
        more = false;
      } else {
        const int stage = (int)(issued % STAGES);
        // the store that last read this stage (STAGES units back) must be done with shared memory
        if (issued >= STAGES) bulk_wait_read<STAGES - LAG - 1>();
        const long long w = u / pieces_per_tile;
        const int off = (int)(u - w * pieces_per_tile) * piece_bytes;
        const Tile t = locate(a, cum, w);
        int len = t.bytes - off;
        if (len > piece_bytes) len = piece_bytes;
        if (len < 0) len = 0;
        pend_len[warp][stage] = len;
        pend_dst[warp][stage] = (GATHER ? t.lin_ptr : t.pool_ptr) + off;
        if (len > 0) {
          const unsigned bar = smem_addr(&bars[warp][stage]);
          mbar_expect_tx(bar, (unsigned)len);
          bulk_load(smem_addr(my_ring + (size_t)stage * piece_bytes), (GATHER ? t.pool_ptr : t.lin_ptr) + off,
                    (unsigned)len, bar);
        }
        ++issued;
      }
    }
    if (issued - stored > LAG || (!more && stored < issued)) {
      const int stage = (int)(stored % STAGES);
      const int len = pend_len[warp][stage];
      if (len > 0) {
        if (!mbar_wait(smem_addr(&bars[warp][stage]), (phase_bits >> stage) & 1u)) { failed = true; break; }
        phase_bits ^= 1u << stage;
        bulk_store(pend_dst[warp][stage], smem_addr(my_ring + (size_t)stage * piece_bytes), (unsigned)len);
      }
      bulk_commit();   // one group per unit, empty or not, so the group arithmetic above holds
      ++stored;
    }
    if (!more && stored == issued) break;
  }
  if (failed) {
    *reinterpret_cast<volatile int *>(a.status) = 1;   // pinned host word, read by the host
    __threadfence_system();
    // give loads still in flight a bounded chance to land before shared memory goes away
    for (int s = 0; s < STAGES; ++s) mbar_wait(smem_addr(&bars[warp][s]), (phase_bits >> s) & 1u);
  }
  bulk_wait_all();
  if (a.stamp) atomicMax(a.stamp + 1, global_ns());                  // every pipeline, after its last store landed
}

// Synthetic competing load: every CTA streams one 32 KiB slice of a large buffer and folds it into a sink word.
// CTAs are short-lived on purpose, so higher-priority mover CTAs get SM slots as these retire.
__global__ void __launch_bounds__(256) read_load_kernel(const uint4 *buf, unsigned long long nvec, unsigned long long *sink) {
  const unsigned long long base = (unsigned long long)blockIdx.x * (256 * 8) + threadIdx.x;
  uint4 v[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const unsigned long long i = base + 256ull * k;
    v[k] = i < nvec ? __ldcs(buf + i) : make_uint4(0, 0, 0, 0);
  }
  unsigned acc = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, d);
  if ((threadIdx.x & 31) == 0) atomicXor(sink + (blockIdx.x & 1023), (unsigned long long)acc);
}

// Self-test of the give-up path: one thread waits, with a small limit, on an mbarrier that nothing will ever
// complete; the wait must run out, the thread records it in the status word and returns.
__global__ void wait_limit_probe_kernel(int *status, unsigned limit) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_addr(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(smem_addr(&bar), 0, limit)) {
      *reinterpret_cast<volatile int *>(status) = 2;
      __threadfence_system();
    }
  }
}

int default_grid(int grid_limit, int sm_count, int ctas_per_sm, long long work_ctas) {
  long long g = (long long)sm_count * ctas_per_sm;
  if (grid_limit > 0 && g > grid_limit) g = grid_limit;
  if (g > work_ctas) g = work_ctas;
  return g < 1 ? 1 : (int)g;
}

template <bool GATHER>
cudaError_t launch_bulk_t(const MoveArgs &a, const BulkShape &sh, int grid, size_t smem, cudaStream_t s) {
  switch (sh.stages) {
    case 2: move_bulk_kernel<GATHER, 2><<<grid, sh.warps * 32, smem, s>>>(a, sh.piece_bytes); break;
    case 3: move_bulk_kernel<GATHER, 3><<<grid, sh.warps * 32, smem, s>>>(a, sh.piece_bytes); break;
    case 4: move_bulk_kernel<GATHER, 4><<<grid, sh.warps * 32, smem, s>>>(a, sh.piece_bytes); break;
    case 6: move_bulk_kernel<GATHER, 6><<<grid, sh.warps * 32, smem, s>>>(a, sh.piece_bytes); break;
    case 8: move_bulk_kernel<GATHER, 8><<<grid, sh.warps * 32, smem, s>>>(a, sh.piece_bytes); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

template <bool GATHER, int STAGES>
cudaError_t opt_in(size_t smem) {
  return cudaFuncSetAttribute(move_bulk_kernel<GATHER, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace

cudaError_t launch_move_warp(bool gather, const MoveArgs &a, int grid_limit, int sm_count, cudaStream_t s) {
  if (a.total_tiles <= 0) return cudaSuccess;
  if (a.nsegs < 1 || a.nsegs > kMaxSegs || !a.work) return cudaErrorInvalidValue;
  static int ctas_per_sm = 0;                     // co-resident CTAs: the grid is one full wave, never more
  if (!ctas_per_sm) {
    int n = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, move_warp_kernel<true>, kWarpThreads, 0);
    if (e != cudaSuccess) return e;
    ctas_per_sm = n > 0 ? n : 1;
  }
  const int warps_per_cta = kWarpThreads / 32;
  const long long work_ctas = (a.total_tiles + warps_per_cta - 1) / warps_per_cta;
  const int grid = default_grid(grid_limit, sm_count, ctas_per_sm, work_ctas);
  const size_t smem = sizeof(long long) * (size_t)(a.nsegs + 1);
  if (gather) move_warp_kernel<true><<<grid, kWarpThreads, smem, s>>>(a);
  else move_warp_kernel<false><<<grid, kWarpThreads, smem, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_read_load(const void *buf, unsigned long long bytes, int launches, void *sink, cudaStream_t s) {
  const unsigned long long nvec = bytes >> 4;
  const unsigned long long ctas = (nvec + 256 * 8 - 1) / (256 * 8);
  if (ctas < 1 || ctas > 0x7fffffffull) return cudaErrorInvalidValue;
  for (int i = 0; i < launches; ++i)
    read_load_kernel<<<(unsigned)ctas, 256, 0, s>>>(static_cast<const uint4 *>(buf), nvec, static_cast<unsigned long long *>(sink));
  return cudaGetLastError();
}

cudaError_t launch_wait_limit_probe(int *status, unsigned limit, cudaStream_t s) {
  wait_limit_probe_kernel<<<1, 32, 0, s>>>(status, limit);
  return cudaGetLastError();
}

cudaError_t bulk_configure(const BulkShape &sh) {
  if (sh.warps < 1 || sh.warps > kMaxBulkWarps || sh.piece_bytes < 16 || sh.piece_bytes % 16) return cudaErrorInvalidValue;
  const size_t smem = (size_t)sh.warps * sh.stages * sh.piece_bytes;
  cudaError_t e = cudaErrorInvalidValue;
  switch (sh.stages) {
    case 2: e = opt_in<true, 2>(smem); if (e == cudaSuccess) e = opt_in<false, 2>(smem); break;
    case 3: e = opt_in<true, 3>(smem); if (e == cudaSuccess) e = opt_in<false, 3>(smem); break;
    case 4: e = opt_in<true, 4>(smem); if (e == cudaSuccess) e = opt_in<false, 4>(smem); break;
    case 6: e = opt_in<true, 6>(smem); if (e == cudaSuccess) e = opt_in<false, 6>(smem); break;
    case 8: e = opt_in<true, 8>(smem); if (e == cudaSuccess) e = opt_in<false, 8>(smem); break;
    default: break;
  }
  return e;
}

cudaError_t launch_move_bulk(bool gather, const MoveArgs &a, const BulkShape &sh, int grid_limit, int sm_count,
                             cudaStream_t s) {
  if (a.total_tiles <= 0) return cudaSuccess;
  if (a.nsegs < 1 || a.nsegs > kMaxSegs || !a.work) return cudaErrorInvalidValue;
  const size_t smem = (size_t)sh.warps * sh.stages * sh.piece_bytes;
  const int pieces_per_tile = (a.tile_bytes + sh.piece_bytes - 1) / sh.piece_bytes;
  const long long units = a.total_tiles * pieces_per_tile;
  const long long work_ctas = (units + sh.warps - 1) / sh.warps;
  const int ctas_per_sm = smem > 110 * 1024 ? 1 : (smem > 72 * 1024 ? 2 : 3);
  const int grid = default_grid(grid_limit, sm_count, ctas_per_sm, work_ctas);
  return gather ? launch_bulk_t<true>(a, sh, grid, smem, s) : launch_bulk_t<false>(a, sh, grid, smem, s);
}

}  // namespace kvr
