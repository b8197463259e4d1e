/*
 * kvr_oracle.c -- see kvr_oracle.h.  TEST INFRASTRUCTURE ONLY.
 *
 * Everything here is the definition written out: one loop level per array
 * axis, one element per innermost iteration, linear searches, arrays that are
 * shifted with memmove.  It is meant to be checked against the paper by eye,
 * not to be fast.
 */
#include "kvr_oracle.h"

#include <stdlib.h>
#include <string.h>

#define ARENA_ALIGN 4096u

typedef struct {
  uint64_t id;
  int32_t state;
  int64_t n_tokens;
  int32_t nb;             /* ceil(n_tokens / BS): logical blocks, shared prefix included */
  int32_t n_shared;       /* leading blocks that are a shared prefix (whole blocks, never moved) */
  int32_t *blocks;        /* ACTIVE / RETAINED: all nb entries; HOST: the n_shared prefix entries it still refers to */
  uint8_t *image;         /* HOST (with_data): the private suffix, tokens [n_shared*BS, n_tokens) */
  uint64_t image_bytes;   /* (n_tokens - n_shared*BS) * bytes_per_token */
  uint64_t arena_off;     /* HOST */
  uint64_t arena_len;     /* image_bytes rounded up to ARENA_ALIGN */
} orc_req;

typedef struct { uint64_t off, len; uint64_t id; } orc_range;

struct orc_pool {
  int32_t L, H, D, e, BS, NB, layout;
  uint64_t bpt;
  int32_t with_data;
  uint8_t *data;
  uint64_t data_bytes;
  int32_t *freeq;          /* freeq[0] is the head */
  int64_t n_free;
  int32_t *refcnt;         /* per block: how many (request, position) references name it; 0 <=> in the free queue */
  orc_req *reqs;
  int64_t n_reqs, cap_reqs;
  orc_range *used;         /* host ranges in use, sorted by offset */
  int64_t n_used, cap_used;
  uint64_t host_capacity;
  orc_stats st;            /* only the monotone counters live here */
};

/* ---- closed forms and index arithmetic ---------------------------------- */

uint64_t orc_bytes_per_token(int32_t layers, int32_t kv_heads, int32_t head_dim, int32_t dtype_bytes) {
  if (layers < 1 || kv_heads < 1 || head_dim < 1 || dtype_bytes < 1) return 0;
  /* Appendix B: layers x kv_heads x head_dim x dtype_bytes x 2 (K and V) */
  return (uint64_t)layers * (uint64_t)kv_heads * (uint64_t)head_dim * (uint64_t)dtype_bytes * 2u;
}

uint64_t orc_pool_offset(int32_t L, int32_t H, int32_t D, int32_t e, int32_t BS, int32_t NB,
                         int32_t l, int32_t kv, int32_t blk, int32_t slot, int32_t h, int32_t d, int32_t byte,
                         int32_t layout) {
  uint64_t i;
  if (layout == ORC_BLOCK_MAJOR) {
    /* pool[NB][L][2][BS][H][D][e]: Horner form of the row-major index */
    i = (uint64_t)blk;
    i = i * (uint64_t)L + (uint64_t)l;
    i = i * 2u + (uint64_t)kv;
  } else {
    /* pool[L][2][NB][BS][H][D][e] */
    i = (uint64_t)l;
    i = i * 2u + (uint64_t)kv;
    i = i * (uint64_t)NB + (uint64_t)blk;
  }
  i = i * (uint64_t)BS + (uint64_t)slot;
  i = i * (uint64_t)H + (uint64_t)h;
  i = i * (uint64_t)D + (uint64_t)d;
  i = i * (uint64_t)e + (uint64_t)byte;
  return i;
}

uint64_t orc_image_offset(int32_t L, int32_t H, int32_t D, int32_t e, int64_t n,
                          int32_t l, int32_t kv, int64_t t, int32_t h, int32_t d, int32_t byte) {
  (void)L;
  /* image[L][2][n][H][D][e] */
  uint64_t i = (uint64_t)l;
  i = i * 2u + (uint64_t)kv;
  i = i * (uint64_t)n + (uint64_t)t;
  i = i * (uint64_t)H + (uint64_t)h;
  i = i * (uint64_t)D + (uint64_t)d;
  i = i * (uint64_t)e + (uint64_t)byte;
  return i;
}

void orc_gather(const uint8_t *pool, uint8_t *image, int32_t L, int32_t H, int32_t D, int32_t e,
                int32_t BS, int32_t NB, const int32_t *bt, int64_t n, int32_t layout) {
  for (int32_t l = 0; l < L; ++l)
    for (int32_t kv = 0; kv < 2; ++kv)
      for (int64_t t = 0; t < n; ++t) {
        int32_t blk = bt[t / BS];
        int32_t slot = (int32_t)(t % BS);
        for (int32_t h = 0; h < H; ++h)
          for (int32_t d = 0; d < D; ++d)
            for (int32_t b = 0; b < e; ++b)
              image[orc_image_offset(L, H, D, e, n, l, kv, t, h, d, b)] =
                  pool[orc_pool_offset(L, H, D, e, BS, NB, l, kv, blk, slot, h, d, b, layout)];
      }
}

void orc_scatter(uint8_t *pool, const uint8_t *image, int32_t L, int32_t H, int32_t D, int32_t e,
                 int32_t BS, int32_t NB, const int32_t *bt, int64_t n, int32_t layout) {
  for (int32_t l = 0; l < L; ++l)
    for (int32_t kv = 0; kv < 2; ++kv)
      for (int64_t t = 0; t < n; ++t) {
        int32_t blk = bt[t / BS];
        int32_t slot = (int32_t)(t % BS);
        for (int32_t h = 0; h < H; ++h)
          for (int32_t d = 0; d < D; ++d)
            for (int32_t b = 0; b < e; ++b)
              pool[orc_pool_offset(L, H, D, e, BS, NB, l, kv, blk, slot, h, d, b, layout)] =
                  image[orc_image_offset(L, H, D, e, n, l, kv, t, h, d, b)];
      }
}

/* ---- pool --------------------------------------------------------------- */

orc_pool *orc_pool_create(int32_t L, int32_t H, int32_t D, int32_t e, int32_t BS, int32_t NB,
                          uint64_t host_capacity, const int32_t *initial_free_order, int32_t with_data,
                          int32_t layout) {
  if (orc_bytes_per_token(L, H, D, e) == 0 || BS < 1 || NB < 1) return NULL;
  if (layout != ORC_LAYER_MAJOR && layout != ORC_BLOCK_MAJOR) return NULL;
  orc_pool *p = (orc_pool *)calloc(1, sizeof(orc_pool));
  if (!p) return NULL;
  p->L = L; p->H = H; p->D = D; p->e = e; p->BS = BS; p->NB = NB; p->layout = layout;
  p->bpt = orc_bytes_per_token(L, H, D, e);
  p->with_data = with_data;
  p->host_capacity = host_capacity;
  p->freeq = (int32_t *)malloc(sizeof(int32_t) * (size_t)NB);
  if (!p->freeq) { free(p); return NULL; }
  if (initial_free_order) {
    /* must be a permutation of [0, NB) */
    uint8_t *seen = (uint8_t *)calloc((size_t)NB, 1);
    int ok = seen != NULL;
    for (int32_t i = 0; ok && i < NB; ++i) {
      int32_t b = initial_free_order[i];
      if (b < 0 || b >= NB || seen[b]) ok = 0; else seen[b] = 1;
    }
    free(seen);
    if (!ok) { free(p->freeq); free(p); return NULL; }
    memcpy(p->freeq, initial_free_order, sizeof(int32_t) * (size_t)NB);
  } else {
    for (int32_t i = 0; i < NB; ++i) p->freeq[i] = i;
  }
  p->n_free = NB;
  p->refcnt = (int32_t *)calloc((size_t)NB, sizeof(int32_t));
  if (!p->refcnt) { free(p->freeq); free(p); return NULL; }
  if (with_data) {
    p->data_bytes = (uint64_t)NB * (uint64_t)BS * p->bpt;
    p->data = (uint8_t *)calloc((size_t)p->data_bytes, 1);
    if (!p->data) { free(p->refcnt); free(p->freeq); free(p); return NULL; }
  }
  return p;
}

void orc_pool_destroy(orc_pool *p) {
  if (!p) return;
  for (int64_t i = 0; i < p->n_reqs; ++i) { free(p->reqs[i].blocks); free(p->reqs[i].image); }
  free(p->reqs); free(p->used); free(p->freeq); free(p->refcnt); free(p->data); free(p);
}

uint8_t *orc_pool_data(orc_pool *p) { return p ? p->data : NULL; }
uint64_t orc_pool_bytes(orc_pool *p) { return p ? p->data_bytes : 0; }

/* ---- small helpers ------------------------------------------------------ */

static orc_req *find_req(orc_pool *p, uint64_t id) {
  for (int64_t i = 0; i < p->n_reqs; ++i) if (p->reqs[i].id == id) return &p->reqs[i];
  return NULL;
}

static int32_t blocks_for(const orc_pool *p, int64_t n_tokens) {
  return (int32_t)((n_tokens + p->BS - 1) / p->BS);
}

/* pop `nb` ids from the head of the free queue into out[] */
static void freeq_pop(orc_pool *p, int32_t nb, int32_t *out) {
  memcpy(out, p->freeq, sizeof(int32_t) * (size_t)nb);
  memmove(p->freeq, p->freeq + nb, sizeof(int32_t) * (size_t)(p->n_free - nb));
  p->n_free -= nb;
}

/* append ids, in the order given, to the tail */
static void freeq_push(orc_pool *p, const int32_t *ids, int32_t nb) {
  memcpy(p->freeq + p->n_free, ids, sizeof(int32_t) * (size_t)nb);
  p->n_free += nb;
}

static uint64_t round_up(uint64_t x) { return (x + (ARENA_ALIGN - 1)) / ARENA_ALIGN * ARENA_ALIGN; }

/* first fit: the lowest offset at which `len` bytes fit between used ranges.
 * Returns 1 and sets *off, or 0 when no gap is large enough. */
static int arena_first_fit(const orc_pool *p, uint64_t len, uint64_t *off) {
  uint64_t cursor = 0;
  for (int64_t i = 0; i < p->n_used; ++i) {
    if (p->used[i].off - cursor >= len) { *off = cursor; return 1; }
    cursor = p->used[i].off + p->used[i].len;
  }
  if (p->host_capacity >= cursor && p->host_capacity - cursor >= len) { *off = cursor; return 1; }
  return 0;
}

static int arena_insert(orc_pool *p, uint64_t off, uint64_t len, uint64_t id) {
  if (p->n_used == p->cap_used) {
    int64_t nc = p->cap_used ? p->cap_used * 2 : 16;
    orc_range *nu = (orc_range *)realloc(p->used, sizeof(orc_range) * (size_t)nc);
    if (!nu) return 0;
    p->used = nu; p->cap_used = nc;
  }
  int64_t pos = 0;
  while (pos < p->n_used && p->used[pos].off < off) ++pos;
  memmove(p->used + pos + 1, p->used + pos, sizeof(orc_range) * (size_t)(p->n_used - pos));
  p->used[pos].off = off; p->used[pos].len = len; p->used[pos].id = id;
  p->n_used += 1;
  return 1;
}

static void arena_remove(orc_pool *p, uint64_t id) {
  for (int64_t i = 0; i < p->n_used; ++i)
    if (p->used[i].id == id) {
      memmove(p->used + i, p->used + i + 1, sizeof(orc_range) * (size_t)(p->n_used - i - 1));
      p->n_used -= 1;
      return;
    }
}

static void drop_host_copy(orc_pool *p, orc_req *r) {
  if (r->arena_len) arena_remove(p, r->id);
  free(r->image); r->image = NULL;
  r->arena_off = 0; r->arena_len = 0;
}

/* take one reference on each id (a block popped from the free queue starts at 1) */
static void ref_blocks(orc_pool *p, const int32_t *ids, int32_t n) {
  for (int32_t i = 0; i < n; ++i) p->refcnt[ids[i]] += 1;
}

/* give up the references blocks[from .. to) of a request, in logical order; a block whose last
 * reference goes joins the free-queue tail (Appendix A: released blocks return to the eviction tail) */
static void unref_blocks(orc_pool *p, const int32_t *blocks, int32_t from, int32_t to) {
  for (int32_t i = from; i < to; ++i) {
    p->refcnt[blocks[i]] -= 1;
    if (p->refcnt[blocks[i]] == 0) freeq_push(p, &blocks[i], 1);
  }
}

/* the request lets go of every block it refers to */
static void drop_blocks(orc_pool *p, orc_req *r) {
  int32_t held = (r->state == ORC_HOST) ? r->n_shared : r->nb;
  unref_blocks(p, r->blocks, 0, held);
  free(r->blocks); r->blocks = NULL;
}

static int64_t private_tokens(const orc_pool *p, const orc_req *r) {
  return r->n_tokens - (int64_t)r->n_shared * p->BS;
}

/* batch result: the most negative status if any is an error, else the largest */
static int32_t fold(int32_t acc, int32_t s) {
  if (s < 0) return (acc < 0 && acc < s) ? acc : s;
  if (acc < 0) return acc;
  return s > acc ? s : acc;
}

/* ---- request lifecycle -------------------------------------------------- */

int32_t orc_request_admit(orc_pool *p, uint64_t id, int64_t n_tokens, int32_t *out_blocks, int32_t cap) {
  if (!p || n_tokens < 0) return ORC_ERR_INVALID_ARG;
  int64_t nb64 = (n_tokens + p->BS - 1) / p->BS;
  if (out_blocks && (int64_t)cap < nb64) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (r && r->state != ORC_EXPIRED) return ORC_ERR_BAD_STATE;
  if (nb64 > p->n_free) { p->st.hbm_full_rejects++; return ORC_HBM_FULL; }
  int32_t nb = blocks_for(p, n_tokens);
  if (!r) {
    if (p->n_reqs == p->cap_reqs) {
      int64_t nc = p->cap_reqs ? p->cap_reqs * 2 : 16;
      orc_req *nr = (orc_req *)realloc(p->reqs, sizeof(orc_req) * (size_t)nc);
      if (!nr) return ORC_ERR_NOMEM;
      p->reqs = nr; p->cap_reqs = nc;
    }
    r = &p->reqs[p->n_reqs++];
    memset(r, 0, sizeof(*r));
    r->id = id;
  }
  r->state = ORC_ACTIVE;
  r->n_tokens = n_tokens;
  r->nb = nb;
  r->image_bytes = (uint64_t)n_tokens * p->bpt;
  r->n_shared = 0;
  r->blocks = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nb ? nb : 1));
  freeq_pop(p, nb, r->blocks);
  ref_blocks(p, r->blocks, nb);
  if (out_blocks) memcpy(out_blocks, r->blocks, sizeof(int32_t) * (size_t)nb);
  return ORC_OK;
}

/* Admission that shares a prefix (Section 2, approval-gated workload: the shared system prefix is reused through
 * prefix caching, "so only the private suffix contributes per-request suspended state").  The new request's first
 * n_shared logical blocks ARE the donor's first n_shared blocks (one more reference each); the rest come from the
 * free-queue head.  Readings (the paper names no mechanism): sharing is by whole blocks -- n_shared*BS tokens must
 * lie inside both the new request and the donor; the donor may be in any state in which it still refers to those
 * blocks (ACTIVE / RETAINED: any of its full blocks; HOST: its own shared prefix). */
int32_t orc_request_admit_sharing(orc_pool *p, uint64_t id, int64_t n_tokens, uint64_t donor_id, int32_t n_shared,
                                  int32_t *out_blocks, int32_t cap) {
  if (!p || n_tokens < 0 || n_shared < 0) return ORC_ERR_INVALID_ARG;
  int64_t nb64 = (n_tokens + p->BS - 1) / p->BS;
  if ((int64_t)n_shared * p->BS > n_tokens) return ORC_ERR_INVALID_ARG;
  if (out_blocks && (int64_t)cap < nb64) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (r && r->state != ORC_EXPIRED) return ORC_ERR_BAD_STATE;
  int32_t *prefix = NULL;
  if (n_shared > 0) {
    if (donor_id == id) return ORC_ERR_INVALID_ARG;
    orc_req *d = find_req(p, donor_id);
    if (!d) return ORC_ERR_UNKNOWN_REQUEST;
    if (d->state == ORC_ACTIVE || d->state == ORC_RETAINED) {
      if ((int64_t)n_shared * p->BS > d->n_tokens) return ORC_ERR_INVALID_ARG;
    } else if (d->state == ORC_HOST) {
      if (n_shared > d->n_shared) return ORC_ERR_INVALID_ARG;
    } else {
      return ORC_ERR_BAD_STATE;            /* a discarded donor refers to nothing */
    }
    prefix = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_shared);
    if (!prefix) return ORC_ERR_NOMEM;
    memcpy(prefix, d->blocks, sizeof(int32_t) * (size_t)n_shared);
  }
  if (nb64 - n_shared > p->n_free) { free(prefix); p->st.hbm_full_rejects++; return ORC_HBM_FULL; }
  int32_t nb = blocks_for(p, n_tokens);
  if (!r) {
    if (p->n_reqs == p->cap_reqs) {
      int64_t nc = p->cap_reqs ? p->cap_reqs * 2 : 16;
      orc_req *nr = (orc_req *)realloc(p->reqs, sizeof(orc_req) * (size_t)nc);
      if (!nr) { free(prefix); return ORC_ERR_NOMEM; }
      p->reqs = nr; p->cap_reqs = nc;
    }
    r = &p->reqs[p->n_reqs++];
    memset(r, 0, sizeof(*r));
    r->id = id;
  }
  r->state = ORC_ACTIVE;
  r->n_tokens = n_tokens;
  r->nb = nb;
  r->n_shared = n_shared;
  r->image_bytes = (uint64_t)(n_tokens - (int64_t)n_shared * p->BS) * p->bpt;
  r->blocks = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nb ? nb : 1));
  if (n_shared) memcpy(r->blocks, prefix, sizeof(int32_t) * (size_t)n_shared);
  free(prefix);
  freeq_pop(p, nb - n_shared, r->blocks + n_shared);
  ref_blocks(p, r->blocks, nb);
  if (out_blocks) memcpy(out_blocks, r->blocks, sizeof(int32_t) * (size_t)nb);
  return ORC_OK;
}

/* Shared-prefix admission for an engine that runs its own allocator: the prefix is the donor's first n_shared
 * blocks as above, and the caller names the private blocks (each free, named once; the other free ids keep
 * their order).  n_shared + n_private must equal ceil(n_tokens / BS). */
int32_t orc_request_admit_sharing_into(orc_pool *p, uint64_t id, int64_t n_tokens, uint64_t donor_id, int32_t n_shared,
                                       const int32_t *private_blocks, int32_t n_private) {
  if (!p || n_tokens < 0 || n_shared < 0 || n_private < 0 || (n_private > 0 && !private_blocks)) return ORC_ERR_INVALID_ARG;
  if ((int64_t)n_shared * p->BS > n_tokens) return ORC_ERR_INVALID_ARG;
  if ((n_tokens + p->BS - 1) / p->BS != (int64_t)n_shared + (int64_t)n_private) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (r && r->state != ORC_EXPIRED) return ORC_ERR_BAD_STATE;
  int32_t nb = n_shared + n_private;
  int32_t *table = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nb ? nb : 1));
  if (!table) return ORC_ERR_NOMEM;
  if (n_shared > 0) {
    if (donor_id == id) { free(table); return ORC_ERR_INVALID_ARG; }
    orc_req *d = find_req(p, donor_id);
    if (!d) { free(table); return ORC_ERR_UNKNOWN_REQUEST; }
    if (d->state == ORC_ACTIVE || d->state == ORC_RETAINED) {
      if ((int64_t)n_shared * p->BS > d->n_tokens) { free(table); return ORC_ERR_INVALID_ARG; }
    } else if (d->state == ORC_HOST) {
      if (n_shared > d->n_shared) { free(table); return ORC_ERR_INVALID_ARG; }
    } else {
      free(table);
      return ORC_ERR_BAD_STATE;
    }
    memcpy(table, d->blocks, sizeof(int32_t) * (size_t)n_shared);
  }
  for (int32_t i = 0; i < n_private; ++i) {
    int found = 0;
    for (int64_t q = 0; q < p->n_free; ++q) if (p->freeq[q] == private_blocks[i]) found = 1;
    for (int32_t j = 0; j < i; ++j) if (private_blocks[j] == private_blocks[i]) found = 0;
    if (!found) { free(table); return ORC_ERR_INVALID_ARG; }
  }
  if (!r) {
    if (p->n_reqs == p->cap_reqs) {
      int64_t nc = p->cap_reqs ? p->cap_reqs * 2 : 16;
      orc_req *nr = (orc_req *)realloc(p->reqs, sizeof(orc_req) * (size_t)nc);
      if (!nr) { free(table); return ORC_ERR_NOMEM; }
      p->reqs = nr; p->cap_reqs = nc;
    }
    r = &p->reqs[p->n_reqs++];
    memset(r, 0, sizeof(*r));
    r->id = id;
  }
  for (int32_t i = 0; i < n_private; ++i)
    for (int64_t q = 0; q < p->n_free; ++q)
      if (p->freeq[q] == private_blocks[i]) {
        memmove(p->freeq + q, p->freeq + q + 1, sizeof(int32_t) * (size_t)(p->n_free - q - 1));
        p->n_free -= 1;
        break;
      }
  if (n_private) memcpy(table + n_shared, private_blocks, sizeof(int32_t) * (size_t)n_private);
  r->state = ORC_ACTIVE;
  r->n_tokens = n_tokens;
  r->nb = nb;
  r->n_shared = n_shared;
  r->image_bytes = (uint64_t)(n_tokens - (int64_t)n_shared * p->BS) * p->bpt;
  r->blocks = table;
  ref_blocks(p, r->blocks, nb);
  return ORC_OK;
}

/* admission into blocks the caller names (an engine with its own allocator mirrors its choice here):
 * every block must be free and named once; the other free ids keep their order */
int32_t orc_request_admit_into(orc_pool *p, uint64_t id, int64_t n_tokens, const int32_t *blocks, int32_t nb) {
  if (!p || n_tokens < 0 || nb < 0 || (nb > 0 && !blocks)) return ORC_ERR_INVALID_ARG;
  if ((n_tokens + p->BS - 1) / p->BS != (int64_t)nb) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (r && r->state != ORC_EXPIRED) return ORC_ERR_BAD_STATE;
  for (int32_t i = 0; i < nb; ++i) {
    int found = 0;
    for (int64_t q = 0; q < p->n_free; ++q) if (p->freeq[q] == blocks[i]) found = 1;
    for (int32_t j = 0; j < i; ++j) if (blocks[j] == blocks[i]) found = 0;
    if (!found) return ORC_ERR_INVALID_ARG;
  }
  if (!r) {
    if (p->n_reqs == p->cap_reqs) {
      int64_t nc = p->cap_reqs ? p->cap_reqs * 2 : 16;
      orc_req *nr = (orc_req *)realloc(p->reqs, sizeof(orc_req) * (size_t)nc);
      if (!nr) return ORC_ERR_NOMEM;
      p->reqs = nr; p->cap_reqs = nc;
    }
    r = &p->reqs[p->n_reqs++];
    memset(r, 0, sizeof(*r));
    r->id = id;
  }
  for (int32_t i = 0; i < nb; ++i)
    for (int64_t q = 0; q < p->n_free; ++q)
      if (p->freeq[q] == blocks[i]) {
        memmove(p->freeq + q, p->freeq + q + 1, sizeof(int32_t) * (size_t)(p->n_free - q - 1));
        p->n_free -= 1;
        break;
      }
  r->state = ORC_ACTIVE;
  r->n_tokens = n_tokens;
  r->nb = nb;
  r->image_bytes = (uint64_t)n_tokens * p->bpt;
  r->n_shared = 0;
  r->blocks = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nb ? nb : 1));
  memcpy(r->blocks, blocks, sizeof(int32_t) * (size_t)nb);
  ref_blocks(p, r->blocks, nb);
  return ORC_OK;
}

int32_t orc_request_release(orc_pool *p, uint64_t id) {
  if (!p) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  if (r->state == ORC_ACTIVE || r->state == ORC_RETAINED) drop_blocks(p, r);
  if (r->state == ORC_HOST) { drop_host_copy(p, r); drop_blocks(p, r); }   /* the copy, and the prefix it still refers to */
  int64_t i = r - p->reqs;
  memmove(p->reqs + i, p->reqs + i + 1, sizeof(orc_req) * (size_t)(p->n_reqs - i - 1));
  p->n_reqs -= 1;
  return ORC_OK;
}

static int32_t retain_one(orc_pool *p, uint64_t id) {
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  if (r->state != ORC_ACTIVE) return ORC_ERR_BAD_STATE;
  r->state = ORC_RETAINED;           /* state 1 of Eq. 1: blocks stay where they are */
  return ORC_OK;
}

static int32_t suspend_one(orc_pool *p, uint64_t id) {
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  if (r->state != ORC_ACTIVE && r->state != ORC_RETAINED) return ORC_ERR_BAD_STATE;
  uint64_t len = round_up(r->image_bytes), off = 0;
  /* Appendix D admission: no room -> not admitted, nobody displaced */
  if (len && !arena_first_fit(p, len, &off)) { p->st.host_full_rejects++; return ORC_HOST_FULL; }
  if (len && !arena_insert(p, off, len, id)) return ORC_ERR_NOMEM;
  if (p->with_data) {
    r->image = (uint8_t *)malloc((size_t)(r->image_bytes ? r->image_bytes : 1));
    if (!r->image) { if (len) arena_remove(p, id); return ORC_ERR_NOMEM; }
    /* only the private suffix is per-request state: the image is the gather over the private part of the table */
    orc_gather(p->data, r->image, p->L, p->H, p->D, p->e, p->BS, p->NB, r->blocks + r->n_shared,
               private_tokens(p, r), p->layout);
  }
  r->arena_off = off; r->arena_len = len;
  /* private blocks are let go in logical order (free tail when the last reference goes); the request keeps
   * referring to its shared prefix, which therefore stays resident while the request waits on the host */
  unref_blocks(p, r->blocks, r->n_shared, r->nb);
  r->state = ORC_HOST;               /* state 2 of Eq. 1 */
  p->st.suspends++; p->st.bytes_suspended += r->image_bytes;
  return ORC_OK;
}

static int32_t expire_one(orc_pool *p, uint64_t id) {
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  if (r->state == ORC_HOST) {
    p->st.bytes_expired_from_host += r->image_bytes;
    drop_host_copy(p, r);
    drop_blocks(p, r);               /* the shared prefix it still referred to */
  } else if (r->state == ORC_ACTIVE || r->state == ORC_RETAINED) {
    drop_blocks(p, r);
  } else {
    return ORC_ERR_BAD_STATE;        /* one-shot: an expired request is not expired again */
  }
  r->state = ORC_EXPIRED;            /* state 3 of Eq. 1: recompute at resume */
  p->st.expires++; p->st.recompute_marked++;
  return ORC_OK;
}

/* `fresh` holds the nb - n_shared ids just taken for the private part (ownership passes to this function) */
static int32_t resume_with_blocks(orc_pool *p, orc_req *r, int32_t *fresh) {
  int32_t n_priv = r->nb - r->n_shared;
  if (p->with_data)
    orc_scatter(p->data, r->image, p->L, p->H, p->D, p->e, p->BS, p->NB, fresh, private_tokens(p, r), p->layout);
  drop_host_copy(p, r);
  ref_blocks(p, fresh, n_priv);
  /* the table is the prefix the request never let go of, followed by the new private blocks */
  int32_t *table = (int32_t *)malloc(sizeof(int32_t) * (size_t)(r->nb ? r->nb : 1));
  if (r->n_shared) memcpy(table, r->blocks, sizeof(int32_t) * (size_t)r->n_shared);
  if (n_priv) memcpy(table + r->n_shared, fresh, sizeof(int32_t) * (size_t)n_priv);
  free(fresh); free(r->blocks);
  r->blocks = table;
  r->state = ORC_ACTIVE;
  p->st.resumes++; p->st.bytes_resumed += r->image_bytes;
  return ORC_OK;
}

static int32_t resume_one(orc_pool *p, uint64_t id) {
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  if (r->state == ORC_RETAINED) { r->state = ORC_ACTIVE; p->st.resident_resumes++; return ORC_RESIDENT; }
  if (r->state == ORC_EXPIRED) return ORC_RECOMPUTE;
  if (r->state != ORC_HOST) return ORC_ERR_BAD_STATE;
  int32_t n_priv = r->nb - r->n_shared;
  if ((int64_t)n_priv > p->n_free) { p->st.hbm_full_rejects++; return ORC_HBM_FULL; }
  int32_t *blocks = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_priv ? n_priv : 1));
  if (!blocks) return ORC_ERR_NOMEM;
  freeq_pop(p, n_priv, blocks);
  return resume_with_blocks(p, r, blocks);
}

int32_t orc_resume_from_host_into(orc_pool *p, uint64_t id, const int32_t *blocks, int32_t nb) {
  if (!p || nb < 0 || (nb > 0 && !blocks)) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  if (r->state != ORC_HOST) return ORC_ERR_BAD_STATE;
  if (nb != r->nb - r->n_shared) return ORC_ERR_INVALID_ARG;      /* the private part is what moves */
  /* every named block must be free, and named once */
  for (int32_t i = 0; i < nb; ++i) {
    int found = 0;
    for (int64_t q = 0; q < p->n_free; ++q) if (p->freeq[q] == blocks[i]) found = 1;
    for (int32_t j = 0; j < i; ++j) if (blocks[j] == blocks[i]) found = 0;
    if (!found) return ORC_ERR_INVALID_ARG;
  }
  /* take them out of the queue; the others keep their order */
  for (int32_t i = 0; i < nb; ++i)
    for (int64_t q = 0; q < p->n_free; ++q)
      if (p->freeq[q] == blocks[i]) {
        memmove(p->freeq + q, p->freeq + q + 1, sizeof(int32_t) * (size_t)(p->n_free - q - 1));
        p->n_free -= 1;
        break;
      }
  int32_t *mine = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nb ? nb : 1));
  if (!mine) return ORC_ERR_NOMEM;
  memcpy(mine, blocks, sizeof(int32_t) * (size_t)nb);
  return resume_with_blocks(p, r, mine);
}

#define BATCH(NAME, ONE)                                                                   \
  int32_t NAME(orc_pool *p, const uint64_t *ids, int32_t n, int32_t *per_req) {            \
    if (!p || n < 0 || (n > 0 && !ids)) return ORC_ERR_INVALID_ARG;                        \
    int32_t acc = ORC_OK;                                                                  \
    for (int32_t i = 0; i < n; ++i) {                                                      \
      int32_t s = ONE(p, ids[i]);                                                          \
      if (per_req) per_req[i] = s;                                                         \
      acc = fold(acc, s);                                                                  \
    }                                                                                      \
    return acc;                                                                            \
  }
BATCH(orc_retain_in_hbm, retain_one)
BATCH(orc_suspend_to_host, suspend_one)
BATCH(orc_expire, expire_one)
BATCH(orc_resume_from_host, resume_one)

/* ---- observation -------------------------------------------------------- */

int32_t orc_request_info(orc_pool *p, uint64_t id, int32_t *state, int64_t *n_tokens, int32_t *nb,
                         int32_t *blocks, int32_t cap, const uint8_t **image, uint64_t *image_bytes,
                         uint64_t *arena_offset) {
  if (!p) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  int held = (r->state == ORC_ACTIVE || r->state == ORC_RETAINED);
  if (state) *state = r->state;
  if (n_tokens) *n_tokens = r->n_tokens;
  if (nb) *nb = r->nb;
  if (blocks && held) {
    if (cap < r->nb) return ORC_ERR_INVALID_ARG;
    memcpy(blocks, r->blocks, sizeof(int32_t) * (size_t)r->nb);
  }
  if (image) *image = (r->state == ORC_HOST) ? r->image : NULL;
  if (image_bytes) *image_bytes = r->image_bytes;
  if (arena_offset) *arena_offset = (r->state == ORC_HOST) ? r->arena_off : 0;
  return ORC_OK;
}

int32_t orc_pool_stats(orc_pool *p, orc_stats *out) {
  if (!p || !out) return ORC_ERR_INVALID_ARG;
  orc_stats s = p->st;
  s.blocks_total = p->NB; s.blocks_free = p->n_free;
  s.blocks_active = s.blocks_pinned = 0;
  s.n_active = s.n_retained = s.n_host = s.n_expired = 0;
  for (int64_t i = 0; i < p->n_reqs; ++i) {
    const orc_req *r = &p->reqs[i];
    if (r->state == ORC_ACTIVE) s.n_active++;
    if (r->state == ORC_RETAINED) s.n_retained++;
    if (r->state == ORC_HOST) s.n_host++;
    if (r->state == ORC_EXPIRED) s.n_expired++;
  }
  /* a block is pinned when a suspended context (RETAINED, or on the host and still referring to its shared prefix)
   * names it; every other held block is active.  Counted per distinct block, by scanning every table. */
  for (int32_t b = 0; b < p->NB; ++b) {
    int held = 0, pinned = 0;
    for (int64_t i = 0; i < p->n_reqs; ++i) {
      const orc_req *r = &p->reqs[i];
      int32_t cnt = (r->state == ORC_ACTIVE || r->state == ORC_RETAINED) ? r->nb : (r->state == ORC_HOST ? r->n_shared : 0);
      for (int32_t k = 0; k < cnt; ++k)
        if (r->blocks[k] == b) { held = 1; if (r->state != ORC_ACTIVE) pinned = 1; }
    }
    if (pinned) s.blocks_pinned++; else if (held) s.blocks_active++;
  }
  s.host_capacity = p->host_capacity; s.host_used = 0; s.host_largest_hole = 0;
  uint64_t cursor = 0;
  for (int64_t i = 0; i < p->n_used; ++i) {
    s.host_used += p->used[i].len;
    uint64_t gap = p->used[i].off - cursor;
    if (gap > s.host_largest_hole) s.host_largest_hole = gap;
    cursor = p->used[i].off + p->used[i].len;
  }
  if (p->host_capacity > cursor && p->host_capacity - cursor > s.host_largest_hole)
    s.host_largest_hole = p->host_capacity - cursor;
  s.host_largest_hole = s.host_largest_hole / ARENA_ALIGN * ARENA_ALIGN;
  *out = s;
  return ORC_OK;
}

int64_t orc_free_queue(orc_pool *p, int32_t *out, int64_t cap) {
  if (!p) return -1;
  if (out) memcpy(out, p->freeq, sizeof(int32_t) * (size_t)(p->n_free < cap ? p->n_free : cap));
  return p->n_free;
}

/* the shared prefix a request refers to (any state but EXPIRED): its length in blocks, and the ids */
int32_t orc_request_sharing(orc_pool *p, uint64_t id, int32_t *n_shared, int32_t *blocks, int32_t cap) {
  if (!p) return ORC_ERR_INVALID_ARG;
  orc_req *r = find_req(p, id);
  if (!r) return ORC_ERR_UNKNOWN_REQUEST;
  int32_t ns = (r->state == ORC_EXPIRED) ? 0 : r->n_shared;
  if (n_shared) *n_shared = ns;
  if (blocks) {
    if (cap < ns) return ORC_ERR_INVALID_ARG;
    if (ns) memcpy(blocks, r->blocks, sizeof(int32_t) * (size_t)ns);
  }
  return ORC_OK;
}

/* number of references to one block (0 = free), -1 for an id out of range */
int32_t orc_block_refcount(orc_pool *p, int32_t blk) {
  if (!p || blk < 0 || blk >= p->NB) return -1;
  return p->refcnt[blk];
}
