/*
 * kvr_oracle.h -- plain, slow, single-threaded CPU statement of the tiered KV
 * retention data path.  TEST INFRASTRUCTURE ONLY: nothing in the product
 * library includes, links or calls this; only the tests, the smoke check and
 * the benchmark's CPU-baseline leg do.  It shares no source with the CUDA
 * library (own structs, own index arithmetic, per-element loops).
 *
 * What the paper fixes and this file restates:
 *   - three retention states per suspended request: 1 = GPU HBM, 2 = host
 *     DRAM, 3 = discarded (Section 3.1, Eq. 1; beta_1 = 0 so a resume from HBM
 *     moves nothing);
 *   - per-token KV bytes = layers x kv_heads x head_dim x dtype_bytes x 2
 *     (Appendix B, price-vector calibration: 80 x 8 x 128 x 2 x 2 = 327,680);
 *   - one-shot expiry of the host copy; host capacity enforced at admission,
 *     a request that finds the tier full is not admitted and residents are
 *     never displaced; expiry frees capacity (Appendix D);
 *   - pinned (retained) blocks stay allocated and are unavailable to others;
 *     released blocks go to the tail of the free queue (Appendix A,
 *     victim-exclusion patch).
 * What the paper leaves open (layout of the paged pool and of the host image,
 * order of the free queue, arena placement rule) is fixed here as:
 *   pool  : bytes [L][2][NB][BS][H][D][e]   (plane 0 = K, plane 1 = V)
 *   image : bytes [L][2][n_tokens][H][D][e] (valid tokens only)
 *   free queue: FIFO (pop head, push tail, in logical block order)
 *   arena : first fit at the lowest offset, sizes rounded up to 4096 bytes.
 *
 * Pins (tests, CPU only): the paper's worked byte counts, numpy fancy-indexing
 * on identity tables, a dictionary-based brute force on pools of <= 6 blocks,
 * round-trip identity under arbitrary relabelling, occupancy arithmetic of
 * Appendix A (42,548-block pool, 525-block contexts, 81 fit); for shared prefixes the
 * paper's 5.4K + 3.0K token split (image = 983,040,000 bytes), conservation with
 * reference counts, and brute force over two requests sharing a prefix.
 * Throughput of this code is a reported baseline only: parity unpinned.
 */
#ifndef KVR_ORACLE_H
#define KVR_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct orc_pool orc_pool;

/* status codes: numerically identical to the library's so logs compare */
enum {
  ORC_OK = 0, ORC_RESIDENT = 1, ORC_RECOMPUTE = 2, ORC_HOST_FULL = 3, ORC_HBM_FULL = 4,
  ORC_ERR_INVALID_ARG = -1, ORC_ERR_UNKNOWN_REQUEST = -2, ORC_ERR_BAD_STATE = -3,
  ORC_ERR_GEOMETRY = -4, ORC_ERR_NOMEM = -7
};
/* request states */
enum { ORC_ACTIVE = 0, ORC_RETAINED = 1, ORC_HOST = 3, ORC_EXPIRED = 5 };

typedef struct {
  int64_t blocks_total, blocks_free, blocks_active, blocks_pinned;
  uint64_t host_capacity, host_used, host_largest_hole;
  int64_t n_active, n_retained, n_host, n_expired;
  int64_t suspends, resumes, resident_resumes, expires, recompute_marked;
  int64_t host_full_rejects, hbm_full_rejects;
  uint64_t bytes_suspended, bytes_resumed, bytes_expired_from_host;
} orc_stats;

/* Pool layouts (the paper names none; both keep one (layer, plane, block) tile contiguous):
 *   ORC_LAYER_MAJOR : bytes [L][2][NB][BS][H][D][e]   (the default reading)
 *   ORC_BLOCK_MAJOR : bytes [NB][L][2][BS][H][D][e]   (all planes of a block adjacent) */
enum { ORC_LAYER_MAJOR = 0, ORC_BLOCK_MAJOR = 1 };

/* Appendix B closed form; 0 when any factor is < 1. */
uint64_t orc_bytes_per_token(int32_t layers, int32_t kv_heads, int32_t head_dim, int32_t dtype_bytes);

/* Byte offset of byte `byte` of element (h, d) of token slot `slot` of block
 * `blk` of plane kv of layer l in the pool array; and of token t in an image
 * of n tokens.  Written from the array declarations above, nothing else. */
uint64_t orc_pool_offset(int32_t L, int32_t H, int32_t D, int32_t e, int32_t BS, int32_t NB,
                         int32_t l, int32_t kv, int32_t blk, int32_t slot, int32_t h, int32_t d, int32_t byte,
                         int32_t layout);
uint64_t orc_image_offset(int32_t L, int32_t H, int32_t D, int32_t e, int64_t n,
                          int32_t l, int32_t kv, int64_t t, int32_t h, int32_t d, int32_t byte);

/* with_data = 0: bookkeeping only (no pool bytes, no images).
 * initial_free_order: permutation of [0, NB) or NULL for identity. */
orc_pool *orc_pool_create(int32_t L, int32_t H, int32_t D, int32_t e, int32_t BS, int32_t NB,
                          uint64_t host_capacity, const int32_t *initial_free_order, int32_t with_data,
                          int32_t layout);
void orc_pool_destroy(orc_pool *);
uint8_t *orc_pool_data(orc_pool *);      /* NULL when with_data = 0 */
uint64_t orc_pool_bytes(orc_pool *);

int32_t orc_request_admit(orc_pool *, uint64_t id, int64_t n_tokens, int32_t *out_blocks, int32_t cap);
int32_t orc_request_admit_into(orc_pool *, uint64_t id, int64_t n_tokens, const int32_t *blocks, int32_t nb);
/* Shared prefix (Section 2: the system prefix is shared through prefix caching and only the private suffix is
 * per-request state).  The new request's first n_shared blocks are the donor's first n_shared blocks, reference
 * counted; a block returns to the free queue when its last reference goes.  While such a request is on the host it
 * keeps its references to the prefix (the prefix stays resident) and its image holds the private suffix only:
 * tokens [n_shared*BS, n_tokens), (n_tokens - n_shared*BS) * bytes_per_token bytes. */
int32_t orc_request_admit_sharing(orc_pool *, uint64_t id, int64_t n_tokens, uint64_t donor_id, int32_t n_shared,
                                  int32_t *out_blocks, int32_t cap);
int32_t orc_request_admit_sharing_into(orc_pool *, uint64_t id, int64_t n_tokens, uint64_t donor_id, int32_t n_shared,
                                       const int32_t *private_blocks, int32_t n_private);
int32_t orc_request_sharing(orc_pool *, uint64_t id, int32_t *n_shared, int32_t *blocks, int32_t cap);
int32_t orc_block_refcount(orc_pool *, int32_t blk);
int32_t orc_request_release(orc_pool *, uint64_t id);
int32_t orc_retain_in_hbm(orc_pool *, const uint64_t *ids, int32_t n, int32_t *per_req);
int32_t orc_suspend_to_host(orc_pool *, const uint64_t *ids, int32_t n, int32_t *per_req);
int32_t orc_expire(orc_pool *, const uint64_t *ids, int32_t n, int32_t *per_req);
int32_t orc_resume_from_host(orc_pool *, const uint64_t *ids, int32_t n, int32_t *per_req);
int32_t orc_resume_from_host_into(orc_pool *, uint64_t id, const int32_t *blocks, int32_t nb);

/* state, token count, block count, block table (ACTIVE/RETAINED), image
 * pointer / bytes / arena offset (HOST).  Any out pointer may be NULL. */
int32_t orc_request_info(orc_pool *, uint64_t id, int32_t *state, int64_t *n_tokens, int32_t *nb,
                         int32_t *blocks, int32_t cap, const uint8_t **image, uint64_t *image_bytes,
                         uint64_t *arena_offset);
int32_t orc_pool_stats(orc_pool *, orc_stats *out);
/* copies the free queue, head first; returns its length */
int64_t orc_free_queue(orc_pool *, int32_t *out, int64_t cap);

/* The two data movements on their own, for timing and for element checks:
 * image[l][kv][t][h][d] = pool[l][kv][bt[t / BS]][t % BS][h][d], and back. */
void orc_gather(const uint8_t *pool, uint8_t *image, int32_t L, int32_t H, int32_t D, int32_t e,
                int32_t BS, int32_t NB, const int32_t *bt, int64_t n, int32_t layout);
void orc_scatter(uint8_t *pool, const uint8_t *image, int32_t L, int32_t H, int32_t D, int32_t e,
                 int32_t BS, int32_t NB, const int32_t *bt, int64_t n, int32_t layout);

#ifdef __cplusplus
}
#endif
#endif
