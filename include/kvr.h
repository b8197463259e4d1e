/*
 * kvr.h -- C ABI of the tiered KV-retention data mover for one GPU.
 *
 * The paper prices three places a suspended request's KV cache can be
 * (Section 3.1, Eq. 1: state 1 = GPU HBM, 2 = host DRAM, 3 = discarded) and a
 * two-stage policy that moves it between them (Section 3.4; exact semantics in
 * Appendix D).  This library is the mechanism under that policy: a paged HBM
 * block pool, a pinned host arena, and the moves between the two.
 *
 *   suspend : gather a request's scattered K/V blocks, by its block table,
 *             into one contiguous image in pinned host memory; free the blocks
 *   resume  : scatter the image into freshly allocated, non-contiguous blocks
 *   retain  : leave the blocks where they are, count them as pinned
 *   expire  : drop the host image (or the blocks); resume then answers
 *             "recompute"
 *
 * Layouts (the paper leaves them open; they are fixed here):
 *   pool  : bytes [layers][2][num_blocks][block_size][kv_heads][head_dim][dtype_bytes]
 *           plane 0 = K, plane 1 = V; one (layer, plane, block) tile is contiguous
 *           (KVR_LAYER_MAJOR, the default); or, with KVR_BLOCK_MAJOR,
 *           bytes [num_blocks][layers][2][block_size][kv_heads][head_dim][dtype_bytes]
 *   image : bytes [layers][2][n_tokens][kv_heads][head_dim][dtype_bytes]
 *           exactly n_tokens * kvr_bytes_per_token() bytes, valid tokens only
 * Bookkeeping rules (also fixed here): the free queue is FIFO (allocate from
 * the head, release to the tail in logical block order); host ranges are
 * placed first-fit at the lowest offset in 4096-byte granules.
 *
 * Conventions
 *   - every pointer argument is a HOST pointer unless its comment says device;
 *   - the pool handle and all metadata belong to the library; buffers passed in
 *     kvr_config belong to the caller and must outlive the pool;
 *   - no exceptions cross this boundary; every call returns a kvr_status:
 *     0 = done, > 0 = a normal outcome the policy must handle, < 0 = error.
 *     Batch calls handle the requests in the order given, each one atomically
 *     (moved or unchanged), write each outcome to per_req (may be NULL) and
 *     return the most negative status if any is an error, else the largest;
 *   - moves are asynchronous: a call enqueues GPU work and returns, unless
 *     KVR_SYNC is given.  Bookkeeping (states, block tables, arena offsets) is
 *     final when the call returns; the bytes are final once kvr_wait() on the
 *     request (or KVR_ALL) returns KVR_OK.  Until then kvr_request_info()
 *     reports KVR_SUSPENDING / KVR_RESUMING (unless a later call has already
 *     changed the settled state, e.g. a resuming request retained again).  Later calls that touch the same
 *     blocks or host bytes are ordered after the move on the device, so the
 *     caller never has to wait for correctness of the library's own moves;
 *   - calls on one pool may come from any thread: they are serialised by a lock inside the pool and make the
 *     pool's device current for their duration.  Whenever a call has to wait on the host for GPU work (kvr_wait,
 *     KVR_SYNC, an expire / release / admit that meets a move in flight, a move call that finds every descriptor
 *     buffer taken) it gives the lock up while it sleeps, so other threads keep working on the pool.
 *     kvr_pool_destroy must not race with other calls.  A kvr_controller is single-threaded;
 *   - a move call that fails while enqueueing (a CUDA error, out of host memory) leaves every request of the batch
 *     exactly as it was: states, block tables, free-queue order, arena ranges and counters are restored, GPU work
 *     already queued for it is waited for, and each affected per_req entry carries the error;
 *   - nothing is allocated on the move path: streams, events of the staging ring, staging memory and the
 *     descriptor buffers (max_moves_in_flight of them, each large enough for the block tables of the whole pool)
 *     exist from kvr_pool_create on.  The one exception is a move whose descriptors exceed such a buffer (tens of
 *     thousands of chunk pieces): it takes a one-off buffer that is freed when the move retires.
 */
#ifndef KVR_H
#define KVR_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvr_pool kvr_pool;
typedef int32_t kvr_status;

enum {
  KVR_OK = 0,
  KVR_RESIDENT = 1,      /* resume of a retained request: nothing moved (beta_1 = 0) */
  KVR_RECOMPUTE = 2,     /* resume of an expired request: caller must re-prefill */
  KVR_HOST_FULL = 3,     /* suspend not admitted to the host tier; request unchanged */
  KVR_HBM_FULL = 4,      /* not enough free blocks; request unchanged */
  KVR_ERR_INVALID_ARG = -1,
  KVR_ERR_UNKNOWN_REQUEST = -2,
  KVR_ERR_BAD_STATE = -3,
  KVR_ERR_GEOMETRY = -4,
  KVR_ERR_CUDA = -5,
  KVR_ERR_TIMEOUT = -6,
  KVR_ERR_NOMEM = -7
};

/* request states as reported by kvr_request_info() */
enum {
  KVR_ACTIVE = 0, KVR_RETAINED = 1, KVR_SUSPENDING = 2, KVR_HOST = 3, KVR_RESUMING = 4, KVR_EXPIRED = 5
};

/* call flags */
#define KVR_SYNC 1u                  /* wait for the enqueued moves before returning */
#define KVR_LOW_LATENCY 2u           /* batched resume, staged route: end a chunk wherever a request ends, so each
                                        request is complete as soon as its own bytes are in (more, smaller launches) */
/* pool flags (kvr_config.flags) */
#define KVR_METADATA_ONLY 1u         /* bookkeeping only: no buffers, no CUDA calls, nothing moves */
#define KVR_PROFILE 2u               /* bracket every mover launch with timing events (gather_ms, scatter_ms) */

#define KVR_ROUTE_AUTO 0             /* staged (the measured winner on B200); mapped when no staging memory can be had
                                        (neither the caller's nor an allocation) and the arena is mapped host memory */
#define KVR_ROUTE_STAGED 1           /* kernel <-> HBM staging ring <-> chunked cudaMemcpyAsync */
#define KVR_ROUTE_MAPPED 2           /* kernel reads / writes the pinned arena directly over the host link */
#define KVR_ROUTE_DMA2D 3            /* no kernel: one strided cudaMemcpy2DAsync per block, pool <-> arena */
#define KVR_KERNEL_WARP 1            /* one warp per tile, 16-byte loads and stores */
#define KVR_KERNEL_BULK 2            /* bulk async copies through a shared-memory ring */

#define KVR_LAYER_MAJOR 0
#define KVR_BLOCK_MAJOR 1

#define KVR_ALL UINT64_MAX

typedef struct {
  int32_t layers, kv_heads, head_dim, dtype_bytes, block_size;
} kvr_geometry;

typedef struct {
  kvr_geometry g;
  int32_t num_blocks;
  int32_t device;                    /* CUDA device ordinal */
  uint64_t host_capacity_bytes;      /* host tier budget */
  uint64_t chunk_bytes;              /* staging slot size: the granule in which staging memory is reused and the
                                        largest single copy over the link; multiple of 4096, at least one tile;
                                        0 = 64 MiB */
  int32_t staging_slots;             /* slots per direction, in [2, 64]; 0 = 32.  Staging memory is one ring of
                                        staging_slots x chunk_bytes per direction (default 2 x 2 GiB, 2.2 % of a
                                        B200's memory; the link runs as fast with less, only the launches get
                                        smaller); one mover launch covers up to staging_slots - 1 consecutive
                                        slots of its ring */
  int32_t route;                     /* KVR_ROUTE_* */
  int32_t kernel;                    /* KVR_KERNEL_*; 0 = KVR_KERNEL_BULK */
  int32_t max_ctas;                  /* cap on the movers' grid (0 = fill the GPU) */
  uint32_t flags;                    /* KVR_METADATA_ONLY | KVR_PROFILE */
  int32_t layout;                    /* KVR_LAYER_MAJOR (0) or KVR_BLOCK_MAJOR */
  void *device_pool;                 /* DEVICE pointer to num_blocks*block_size*bytes_per_token bytes,
                                        256-byte aligned, or NULL: the library allocates and frees it */
  void *host_arena;                  /* page-locked HOST pointer to host_capacity_bytes bytes, 256-byte
                                        aligned, or NULL: the library allocates and frees it.  A DEVICE
                                        pointer is accepted too (this GPU's memory, or a peer's with peer
                                        access enabled): the tier then lives in HBM and images are device
                                        memory; with KVR_ROUTE_MAPPED the movers write it directly */
  const int32_t *initial_free_order; /* permutation of [0, num_blocks) or NULL = 0, 1, 2, ... */
  /* Everything below may be left zero. */
  void *device_staging;              /* DEVICE pointer to 2 x staging_slots x chunk_bytes bytes, 256-byte aligned
                                        (an engine that owns all of HBM carves it out of its own memory), or NULL:
                                        the library allocates it at pool creation */
  void *streams[4];                  /* cudaStream_t for the gather kernel, the device-to-host copies, the
                                        host-to-device copies and the scatter kernel, in that order; four distinct
                                        streams of cfg->device, or NULL each: the library creates high-priority
                                        non-blocking streams.  Caller-owned streams must not be used for anything
                                        that waits on this pool's moves from inside the same stream */
  uint64_t suspend_single_bytes;     /* a suspend of up to this many bytes is one mover launch; a larger one keeps
                                        its first launch down to one slot, so the link starts at once, and makes
                                        every other launch as large as the ring allows.  0 = 1 GiB: the blocks of
                                        such a request are free 0.35 ms later than they could be, 2 % of the
                                        19 ms the move spends on the link */
  uint64_t resume_single_bytes;      /* the same for a resume, whose last launch is the one kept down to a slot, so
                                        that little scattering remains after the last byte has arrived.  0 =
                                        256 MiB: at most 85 us between the last byte and the request being usable */
  uint64_t copy_piece_bytes;         /* link copies are issued in pieces of at most this size (and never across a
                                        staging slot unless it is larger than a slot); 0 = 64 MiB */
  int32_t max_moves_in_flight;       /* descriptor buffers created with the pool, one per move in flight, in
                                        [1, 256]; 0 = 16.  A move call waits (bounded) while all are taken */
  int32_t bulk_warps, bulk_stages, bulk_piece_bytes;   /* shape of the bulk mover: pipelines per CTA (1..8),
                                        shared-memory stages per pipeline (2, 3, 4, 6 or 8), bytes per bulk copy
                                        (multiple of 16); all three 0 = chosen from the tile size */
} kvr_config;

typedef struct {
  int64_t blocks_total, blocks_free, blocks_active, blocks_pinned;   /* distinct blocks: pinned = named by a RETAINED
                                                     request or by the kept prefix of a HOST request; active = held otherwise */
  uint64_t host_capacity, host_used, host_largest_hole;
  int64_t n_active, n_retained, n_host, n_expired;
  int64_t suspends, resumes, resident_resumes, expires, recompute_marked;
  int64_t host_full_rejects, hbm_full_rejects;
  uint64_t bytes_suspended, bytes_resumed, bytes_expired_from_host;
  /* engine counters (zero for a metadata-only pool) */
  int64_t ops_in_flight;
  int64_t gather_launches, scatter_launches;     /* kernel launches so far */
  int64_t d2h_copies, h2d_copies;                /* cudaMemcpyAsync calls so far */
  uint64_t gather_bytes, scatter_bytes;          /* payload bytes moved by the kernels */
  uint64_t d2h_bytes, h2d_bytes;                 /* bytes moved by copies (descriptors excluded) */
  uint64_t desc_bytes;                           /* descriptor and block-table bytes uploaded */
  double gather_ms, scatter_ms;                  /* summed kernel durations by CUDA events, KVR_PROFILE only */
  double gather_kernel_ms, scatter_kernel_ms;    /* the same launches timed by the kernels themselves (first CTA
                                                    start to last CTA end, %globaltimer), KVR_PROFILE only */
} kvr_stats;

/*
 * Per-token KV bytes = 2 (K and V) x layers x kv_heads x head_dim x dtype_bytes
 * (Appendix B, price-vector calibration: 80 x 8 x 128 x 2 x 2 = 327,680).
 * Returns 0 for a NULL or invalid geometry (any field < 1, dtype_bytes not in
 * {1,2,4}, or kv_heads*head_dim*dtype_bytes not a multiple of 16).
 */
uint64_t kvr_bytes_per_token(const kvr_geometry *g);

/*
 * Create the HBM block pool and the host tier (Appendix A: paged block pool with
 * a free queue; Appendix D: host tier with a capacity enforced at admission).
 * Allocates the staging rings, streams and events on cfg->device, and whichever
 * of device_pool / host_arena is NULL.  *out is set only on KVR_OK.
 * Errors: KVR_ERR_INVALID_ARG (NULL, bad sizes, free order not a permutation),
 * KVR_ERR_GEOMETRY, KVR_ERR_NOMEM, KVR_ERR_CUDA.
 */
kvr_status kvr_pool_create(const kvr_config *cfg, kvr_pool **out);
/* Waits for all moves in flight, then frees everything the library allocated. */
kvr_status kvr_pool_destroy(kvr_pool *pool);

/*
 * Bring a request into the pool as ACTIVE with ceil(n_tokens/block_size) blocks
 * from the head of the free queue (in a server the engine's own allocator does
 * this; here it is what tests and benchmarks use).  out_blocks (cap entries,
 * may be NULL) receives the block table.  The blocks are safe to write when the
 * call returns: it waits for any gather still reading them.  Re-admitting an
 * EXPIRED id is allowed (the recompute happened).  n_tokens = 0 is legal.
 * KVR_HBM_FULL, KVR_ERR_BAD_STATE (id exists), KVR_ERR_INVALID_ARG.
 */
kvr_status kvr_request_admit(kvr_pool *pool, uint64_t req_id, int64_t n_tokens, int32_t *out_blocks, int32_t cap);
/* Same, into blocks the caller names (an engine with its own allocator mirrors its choice): nb =
 * ceil(n_tokens/block_size) ids, each currently free, no repeats; the other free ids keep their order. */
kvr_status kvr_request_admit_into(kvr_pool *pool, uint64_t req_id, int64_t n_tokens, const int32_t *blocks, int32_t nb);
/* Forget a request in any state; its references to blocks are dropped (a block whose last reference goes joins the
 * free tail), its host range is freed. */
kvr_status kvr_request_release(kvr_pool *pool, uint64_t req_id);

/*
 * Shared prefix (Section 2, approval-gated workload: a system prefix shared through prefix caching, so that only
 * the private suffix is per-request suspended state; Appendix B prices that suffix).  The new request's first
 * n_shared_blocks logical blocks ARE the donor's first n_shared_blocks blocks, one more reference each; the rest
 * come from the head of the free queue.  Blocks are reference counted: a block rejoins the free queue only when
 * the last request naming it lets go, so a prefix lives exactly as long as somebody refers to it.  A request keeps
 * referring to its shared prefix while it is RETAINED or on the HOST (the prefix stays resident and is counted in
 * blocks_pinned); kvr_suspend_to_host moves only the private suffix -- tokens [n_shared_blocks * block_size,
 * n_tokens), an image of (n_tokens - n_shared_blocks * block_size) * bytes_per_token bytes -- and a resume gives
 * the request its old prefix followed by fresh blocks.
 * Sharing is by whole blocks: n_shared_blocks * block_size tokens must lie inside the new request and inside the
 * donor.  The donor may be ACTIVE or RETAINED (any of its full blocks) or on the HOST (its own shared prefix);
 * with n_shared_blocks = 0 the donor is ignored and the call equals kvr_request_admit.
 * KVR_HBM_FULL, KVR_ERR_BAD_STATE (id exists, donor EXPIRED), KVR_ERR_UNKNOWN_REQUEST (donor), KVR_ERR_INVALID_ARG.
 */
kvr_status kvr_request_admit_sharing(kvr_pool *pool, uint64_t req_id, int64_t n_tokens, uint64_t donor_id,
                                     int32_t n_shared_blocks, int32_t *out_blocks, int32_t cap);
/* The same for an engine that runs its own allocator: the prefix comes from the donor, the private blocks are named
 * by the caller (n_private ids, each currently free, no repeats; the other free ids keep their order);
 * n_shared_blocks + n_private must equal ceil(n_tokens / block_size). */
kvr_status kvr_request_admit_sharing_into(kvr_pool *pool, uint64_t req_id, int64_t n_tokens, uint64_t donor_id,
                                          int32_t n_shared_blocks, const int32_t *private_blocks, int32_t n_private);
/* The shared prefix a request refers to: its length in blocks and (cap entries, may be NULL) the ids. */
kvr_status kvr_request_sharing(kvr_pool *pool, uint64_t req_id, int32_t *n_shared_blocks, int32_t *blocks, int32_t cap);
/* Number of references to one block (0 = free); -1 for an id out of range. */
int32_t kvr_block_refcount(kvr_pool *pool, int32_t block);

/*
 * State 1 of Eq. 1 (Section 3.1): keep the KV in HBM.  ACTIVE -> RETAINED; the
 * blocks stay allocated and are counted in blocks_pinned (Appendix A, victim
 * exclusion).  No data moves.  Other states: KVR_ERR_BAD_STATE.
 */
kvr_status kvr_retain_in_hbm(kvr_pool *pool, const uint64_t *req, int32_t n, kvr_status *per_req);

/*
 * State 1 -> 2 (Section 3.4 stage one; Appendix D: "on suspension, a context
 * moves to host DRAM").  For each ACTIVE or RETAINED request, in order: reserve
 * an image range in the host arena (no room: KVR_HOST_FULL, request unchanged,
 * nobody displaced -- the replay admission rule of Appendix D), gather
 *   image[l][kv][t][..] = pool[l][kv][table[t / block_size]][t % block_size][..]
 * into it, and append the blocks to the free-queue tail.  Pool bytes are not
 * scrubbed.  flags: KVR_SYNC.
 */
kvr_status kvr_suspend_to_host(kvr_pool *pool, const uint64_t *req, int32_t n, uint32_t flags, kvr_status *per_req);

/*
 * State 2 or 1 -> 3 (Appendix D: when the one-shot timer fires the host copy is
 * discarded, which frees host capacity).  HOST: the image range is freed.
 * ACTIVE / RETAINED: the blocks go to the free tail.  The request becomes
 * EXPIRED and is counted in recompute_marked.  An EXPIRED request cannot be
 * expired again (KVR_ERR_BAD_STATE).  No data moves.
 */
kvr_status kvr_expire(kvr_pool *pool, const uint64_t *req, int32_t n, kvr_status *per_req);

/*
 * Resume (Section 3.1: pays beta_2 from host, nothing from HBM, beta_3 after a
 * discard).  HOST: take ceil(n_tokens/block_size) blocks from the free-queue
 * head (too few: KVR_HBM_FULL, unchanged), scatter the image into them (bytes
 * of a partial last block beyond n_tokens are not written), free the host
 * range, -> ACTIVE.  RETAINED: -> ACTIVE, same blocks, KVR_RESIDENT.  EXPIRED:
 * KVR_RECOMPUTE, unchanged.  ACTIVE: KVR_ERR_BAD_STATE.  flags: KVR_SYNC, KVR_LOW_LATENCY.
 */
kvr_status kvr_resume_from_host(kvr_pool *pool, const uint64_t *req, int32_t n, uint32_t flags, kvr_status *per_req);
/*
 * Same move for one HOST request into blocks the caller names (each currently
 * free, no repeats, nb = its private block count: all of its blocks unless it
 * shares a prefix); the other free ids keep their order.  This is how "any
 * block relabelling" is exercised.
 */
kvr_status kvr_resume_from_host_into(kvr_pool *pool, uint64_t req, const int32_t *blocks, int32_t nb, uint32_t flags);

/*
 * The two kernels on their own, HBM to HBM, no state change: write the images
 * of n ACTIVE/RETAINED requests one after another (each start rounded up to 256
 * bytes) into the DEVICE buffer dst, or read them back from src into the
 * requests' current blocks.  offsets (n entries, may be NULL) receives each
 * image's byte offset.  KVR_ERR_INVALID_ARG if capacity is too small.
 * Used to measure and to check the gather / scatter kernels in isolation.
 */
kvr_status kvr_export_to_device(kvr_pool *pool, const uint64_t *req, int32_t n, void *dst_device,
                                uint64_t capacity, uint64_t *offsets, uint32_t flags);
kvr_status kvr_import_from_device(kvr_pool *pool, const uint64_t *req, int32_t n, const void *src_device,
                                  uint64_t capacity, uint64_t *offsets, uint32_t flags);

/*
 * The paper has no counterpart to this call; it exists for integration.  Some callers cannot allocate
 * device memory: a serving engine that has given all of HBM to its own block allocator, or a
 * latency-critical path that must not hit the device-wide synchronisation an allocation implies.
 * This is kvr_export_to_device for ONE request without a pool handle and without any allocation: the
 * segment record and the block table the gather kernel reads are copied into a fixed array in the
 * library's device image (about 256 KiB, held by every GPU that loads the library until exit), so a
 * request may have at most KVR_NOALLOC_MAX_BLOCKS blocks; more is rejected with KVR_ERR_INVALID_ARG
 * and a message that names the limit.
 *   device_pool : DEVICE, layout of the pool above, 16-byte aligned
 *   block_table : HOST, nb = ceil(n_tokens / block_size) ids in [0, num_blocks)
 *   dst_device  : DEVICE, n_tokens * kvr_bytes_per_token(g) bytes, 16-byte aligned
 *   stream      : cudaStream_t (NULL = default stream); the work is enqueued, not waited for
 * block_table may be pageable or page-locked: it is read only during the call (it is copied to a fixed host-side
 * twin of the array, range-checked there and uploaded from there), so the caller may change or free it as soon
 * as the call returns.  That upload comes from pageable memory, so the call can block the host until the work
 * already queued on `stream` has finished (for instance the previous call's gather).
 * A geometry whose tile (block_size x kv_heads x head_dim x dtype_bytes) exceeds 1 GiB is KVR_ERR_GEOMETRY, as in
 * kvr_pool_create.
 * Runs on the current device.  The first call on each device looks up the array's address; make that
 * call before starting any stream capture.  All calls share the array: calls whose GPU work may overlap
 * (different streams or threads) race on it -- keep them on one stream or wait in between.  Nothing in
 * the array needs clearing: each call overwrites what it uses.
 */
#define KVR_NOALLOC_MAX_BLOCKS 65536
/* (the pool is taken to be KVR_LAYER_MAJOR) */
kvr_status kvr_gather_noalloc(const void *device_pool, const kvr_geometry *g, int32_t num_blocks,
                              const int32_t *block_table, int32_t nb, int64_t n_tokens,
                              void *dst_device, void *stream);

/*
 * Observe one request.  Any out pointer may be NULL.  blocks (cap entries) is
 * written for requests that hold blocks; host_image is a borrowed pointer into
 * the arena, valid while the request stays in HOST; arena_offset is its offset.
 */
kvr_status kvr_request_info(kvr_pool *pool, uint64_t req, int32_t *state, int64_t *n_tokens, int32_t *nb,
                            int32_t *blocks, int32_t cap, const void **host_image, uint64_t *image_bytes,
                            uint64_t *arena_offset);
/*
 * Time the last move of a request took: host_ms from call entry until its work
 * was enqueued, device_ms from the first enqueued work of that call until this
 * request's last byte landed.  KVR_ERR_BAD_STATE if it never moved or the move
 * is still in flight.
 */
kvr_status kvr_request_latency(kvr_pool *pool, uint64_t req, double *host_ms, double *device_ms);

/*
 * Wait until the moves of one request (or KVR_ALL) are complete; polls, never
 * blocks longer than timeout_ms (< 0 = 60 s): KVR_ERR_TIMEOUT.  Surfaces a
 * device-side mover error (a bounded wait that ran out) as KVR_ERR_CUDA.
 */
kvr_status kvr_wait(kvr_pool *pool, uint64_t req_or_all, int64_t timeout_ms);

/*
 * Benchmark support, not part of the method: the synthetic competing load of the long-context interference
 * measurement.  Enqueues `launches` kernels on `stream` (a cudaStream_t), each streaming the DEVICE buffer
 * (bytes, 16-byte aligned) once out of HBM in short-lived CTAs; device_sink is 8 KiB of DEVICE memory the
 * kernels fold what they read into.  Returns at once; time it with events on `stream`.
 */
kvr_status kvr_read_load(const void *device_buf, uint64_t bytes, int32_t launches, void *device_sink, void *stream);

/*
 * The copy benchmark behind the host-resume price beta_2 (Appendix B: one contiguous payload between page-locked
 * host memory and the device, synchronised before and after, repeated): copies `bytes` (clipped to the arena)
 * between the pool's own arena and the pool's staging memory (a temporary device buffer only when `bytes` exceeds
 * it or the pool has none), reps times each way after two warm-ups, and reports
 * the best rate per direction in GB/s (1e9).  This is the link roofline the moves are judged against, measured
 * on the very memory they use.  The arena must hold no image (KVR_ERR_BAD_STATE otherwise): it is overwritten.
 */
kvr_status kvr_probe_link(kvr_pool *pool, uint64_t bytes, int32_t reps, double *d2h_gbs, double *h2d_gbs);

/*
 * Self-test of the movers' give-up path (no counterpart in the paper).  Every wait inside the bulk mover is bounded;
 * when one runs out the kernel writes the pool's device-error word and returns, and kvr_wait() then reports
 * KVR_ERR_CUDA.  This call makes a wait run out on purpose and safely: one thread polls, 4096 times, a barrier that
 * nothing completes.  KVR_OK means the thread gave up and the word was written.  With leave_error_set != 0 the word
 * stays set so that the reporting through kvr_wait() can be observed; kvr_clear_device_error() resets it.
 */
kvr_status kvr_selftest_bounded_wait(kvr_pool *pool, int32_t leave_error_set);
/*
 * Self-test of the movers' table check (no counterpart in the paper).  Every block table is validated on the host
 * before it is uploaded; the kernels check each entry once more against the pool's block count, skip a tile whose
 * entry is out of range and write 3 to the device-error word, so the pool is never addressed outside its extent.
 * This call makes the check fire safely: it launches the gather over one tile whose entry names the pool's last
 * block while telling the kernel that the pool is one block shorter (the entry is out of range for the kernel, yet
 * inside the real allocation).  KVR_OK means the tile was skipped and the word was written.
 */
kvr_status kvr_selftest_block_check(kvr_pool *pool, int32_t leave_error_set);
kvr_status kvr_clear_device_error(kvr_pool *pool);

kvr_status kvr_pool_stats(kvr_pool *pool, kvr_stats *out);

/*
 * The policy that decides when the moves above happen (host code, no GPU work; all times in seconds, costs in
 * GPU-seconds).  kvr_prices is the platform's calibrated price vector (Section 3.2): alpha1 = HBM holding cost per
 * second, beta2 = host-resume cost, beta3 = recomputation cost; valid iff alpha1 > 0 and beta3 > beta2 >= 0.
 */
typedef struct { double alpha1, beta2, beta3; } kvr_prices;
/* Eq. 2: t_1 = beta2 / alpha1 (HBM vs host break-even), t* = beta3 / alpha1 (HBM vs discard). */
kvr_status kvr_policy_break_evens(const kvr_prices *p, double *t1, double *t_star);
/* Eq. 3: lambda_crit = c2 / w_ref; alpha2 = max(0, lambda - lambda_crit) * beta3 / c2; t2 = (beta3 - beta2) / alpha2,
 * +infinity at or below lambda_crit.  c2 = contexts that fit in the host tier.  Either out pointer may be NULL. */
kvr_status kvr_policy_host_ttl(const kvr_prices *p, double lambda, double c2, double w_ref, double *alpha2, double *t2);
/* Measured-cost replay (Appendix D): contexts arrive at arrive[i] (non-decreasing) and wait wait[i]; each is
 * admitted iff one of c2 slots is free, residents are never displaced; a slot is held until the resume or until
 * ttl after arrival (one-shot timer, +infinity = host-retain).  A resume that finds its copy costs beta2, any other
 * beta3.  Outputs: mean cost per request and the fraction resumed from the host copy. */
kvr_status kvr_policy_replay(const kvr_prices *p, const double *arrive, const double *wait, int64_t n, int64_t c2,
                             double ttl, double *mean_cost, double *from_host);
/* Controller (Section 3.4): replay a calibration sample under host-retain and under cpu_ttl(lambda), report both
 * costs and the timer, and set *use_ttl to 1 iff expiration is strictly cheaper.  Out pointers may be NULL. */
kvr_status kvr_policy_select(const kvr_prices *p, const double *arrive, const double *wait, int64_t n, double lambda,
                             int64_t c2, double w_ref, int32_t *use_ttl, double *cost_retain, double *cost_ttl, double *t2);

/*
 * Live controller (Section 3.4 and the live-controller rules of Appendix D), host code on top of the calls above.
 * It keeps a clock the caller advances (seconds, never backwards).  At a suspension the context is pinned in HBM
 * (kvr_retain_in_hbm) and, after hbm_grace_s (0 = at once: t_1 is about a second), moved to the host tier; under
 * KVR_BRANCH_TTL it then gets a one-shot timer t_2(lambda) counted from the offload.  When the host tier is full,
 * KVR_ADMIT_REPLAY discards the newcomer (residents are never displaced) and KVR_ADMIT_LIVE first discards the
 * host copy that has been suspended longest.  gpu_cost accumulates Eq. 1: alpha1 x seconds spent pinned in HBM,
 * beta2 per resume from the host copy, beta3 per resume that must recompute.
 */
typedef struct kvr_controller kvr_controller;
#define KVR_BRANCH_RETAIN 0
#define KVR_BRANCH_TTL 1
#define KVR_ADMIT_REPLAY 0
#define KVR_ADMIT_LIVE 1
typedef struct {
  kvr_prices prices;
  double lambda;             /* offered rate of suspensions, per second */
  double c2;                 /* contexts the host tier holds; <= 0: host capacity / mean_image_bytes */
  double mean_image_bytes;
  double w_ref;              /* reference wait, seconds */
  double hbm_grace_s;
  int32_t branch;            /* KVR_BRANCH_* (kvr_controller_calibrate overrides it) */
  int32_t admission;         /* KVR_ADMIT_* */
} kvr_controller_config;
typedef struct {
  int64_t suspended, offloaded, not_admitted, ttl_expired, evicted_lru;
  int64_t resumed_host, resumed_hbm, recomputed, tracked;
  double gpu_cost, t2;
  int32_t branch, reserved;
} kvr_controller_stats;
kvr_status kvr_controller_create(kvr_pool *pool, const kvr_controller_config *cfg, kvr_controller **out);
kvr_status kvr_controller_destroy(kvr_controller *c);
/* replay the calibration sample under both branches and freeze the cheaper one (kvr_policy_select) */
kvr_status kvr_controller_calibrate(kvr_controller *c, const double *arrive, const double *wait, int64_t n, int32_t *branch);
/* the ACTIVE request `req` suspends at time now: KVR_OK (on the host), KVR_RESIDENT (pinned in HBM for the grace
 * period), KVR_HOST_FULL (not admitted: discarded, it will recompute) */
kvr_status kvr_controller_suspend(kvr_controller *c, uint64_t req, double now);
/* fire every offload and expiry due by `now`; counts may be NULL */
kvr_status kvr_controller_advance(kvr_controller *c, double now, int32_t *n_offloaded, int32_t *n_expired);
/* the request resumes at time now: KVR_OK (restored from host), KVR_RESIDENT, KVR_RECOMPUTE (caller re-admits and
 * prefills), KVR_HBM_FULL (nothing changed; free blocks and call again) */
kvr_status kvr_controller_resume(kvr_controller *c, uint64_t req, double now);
kvr_status kvr_controller_get_stats(kvr_controller *c, kvr_controller_stats *out);

/*
 * Host-made failures for tests (no counterpart in the paper; nothing here touches the GPU).  kind 0: the n-th CUDA
 * runtime call a move makes from now on (event record, stream wait, copy, kernel launch, ...) reports failure
 * WITHOUT being issued; kind 1: the n-th host allocation point of the move path throws as if memory had run out.
 * n = 0 disarms.  kvr_test_points() returns how many such points were passed since the last arming, so a test can
 * walk n over a whole move.
 */
#define KVR_FAIL_CUDA 0
#define KVR_FAIL_ALLOC 1
kvr_status kvr_test_fail_nth(kvr_pool *pool, int32_t kind, int64_t n);
int64_t kvr_test_points(kvr_pool *pool, int32_t kind);

/*
 * The staged route's planner on its own, for tests (no counterpart in the paper; pure host code).  Plans one move of
 * n_items requests of n_tokens[i] tokens through a ring of `slots` slots of slot_bytes, of which one launch may
 * cover launch_slots, starting at slot ring_next; resume != 0 plans a resume (flags: KVR_LOW_LATENCY); the
 * single-launch thresholds may be 0 for the defaults.  Images are laid out one after another from offset 0 in
 * 4096-byte granules.  Outputs (cap records each): chunks -- 6 numbers per launch: first slot, slots, payload bytes,
 * copies, first segment, segments; copies -- 5 per link copy: launch, offset in the arena, offset in the ring,
 * position inside the launch (unused bytes at the ring's end included), bytes; segs -- 5 per segment: byte offset of
 * the request's block table among the tables, where image byte 0 would lie relative to the ring's base, first tile,
 * tiles, blocks of the request; counts -- launches, copies, segments, the ring's next slot afterwards.
 */
kvr_status kvr_test_plan(const kvr_geometry *g, const int64_t *n_tokens, int32_t n_items, uint64_t slot_bytes, int32_t slots,
                         int32_t launch_slots, int32_t ring_next, int32_t resume, uint32_t flags, uint64_t suspend_single_bytes,
                         uint64_t resume_single_bytes, int64_t *chunks, int64_t *copies, int64_t *segs, int64_t cap, int64_t *counts);

/*
 * Placement of the library's own arena (no counterpart in the paper).  Host DRAM is shared between the GPUs of a
 * node; each pool's arena is faulted in by threads bound to the CPUs of the NUMA node its GPU hangs off, so the
 * pages land next to that GPU's link.  kvr_pool_numa_node: the node used (-1: unknown, single-node host, caller's
 * arena).  kvr_numa_lookup: the parsing on its own -- node of the PCI device `pci_bus_id` ("0000:1b:00.0") and the
 * CPUs of that node under `sysfs_root` (NULL = "/sys"); returns the CPU count (cpus: cap entries, may be NULL),
 * *node = -1 and 0 when the tree does not say.
 */
int32_t kvr_pool_numa_node(kvr_pool *pool);
int32_t kvr_numa_lookup(const char *sysfs_root, const char *pci_bus_id, int32_t *node, int32_t *cpus, int32_t cap);

/* copies the free queue, head first, into out (cap entries, may be NULL); returns its length */
int64_t kvr_free_queue(kvr_pool *pool, int32_t *out, int64_t cap);
/* the DEVICE pool pointer and the HOST arena pointer in use (caller's or the library's) */
void *kvr_pool_device_ptr(kvr_pool *pool);
void *kvr_pool_host_arena(kvr_pool *pool);
/* message of the last error on this thread ("" if none) */
const char *kvr_last_error(void);

#ifdef __cplusplus
}
#endif
#endif
