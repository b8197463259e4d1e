// C ABI of the KV retention mover: argument checks and bookkeeping of every entry point.  Each batch call settles
// the bookkeeping at once (states, block tables, arena offsets: the same answers a synchronous implementation
// gives) and hands the byte movement to the transfer engine (kvr_engine.cu), which queues it on the streams.
#include "kvr_pool.hpp"

using namespace kvr;

namespace {

kvr_status check_pool(kvr_pool *p) { return p ? KVR_OK : fail(KVR_ERR_INVALID_ARG, "pool is NULL"); }

// Held for the length of an entry point: serialises callers on the pool and makes the pool's device current
// on the calling thread (putting the caller's device back on the way out).
struct Enter {
  std::unique_lock<std::mutex> lock;
  int prev = -1;
  explicit Enter(kvr_pool *p) : lock(p->mu) {
    if (p->meta_only) return;
    int cur = -1;
    if (cudaGetDevice(&cur) == cudaSuccess && cur != p->device && cudaSetDevice(p->device) == cudaSuccess) prev = cur;
  }
  ~Enter() { if (prev >= 0) cudaSetDevice(prev); }
};

// A descriptor buffer reserved for the length of a move call.  Taking one is the only place where a move call may
// have to wait for earlier moves (all max_moves_in_flight buffers taken); it happens before the call looks at any
// request, because the lock is given up during that wait.
struct DescLease {
  kvr_pool *p;
  int idx = -1;
  explicit DescLease(kvr_pool *pool) : p(pool) {}
  kvr_status take(std::unique_lock<std::mutex> &lock) {
    if (p->meta_only) return KVR_OK;
    const auto t0 = Clock::now();
    for (;;) {
      if (kvr_status s = poll(p)) return s;
      for (size_t i = 0; i < p->descs.size(); ++i)
        if (p->descs[i].h && !p->descs[i].busy && !p->descs[i].one_off) { p->descs[i].busy = kLeased; idx = (int)i; return KVR_OK; }
      if (p->ops.empty()) return KVR_OK;            // every buffer leased by other threads: enqueue falls back to a one-off buffer
      if (ms_since(t0) > 60000.0) return fail(KVR_ERR_TIMEOUT, "every descriptor buffer is still taken after 60 s");
      const uint64_t oldest = p->ops.begin()->first;
      const kvr_status s = wait_unlocked(p, lock, oldest, false, 60000);
      if (s != KVR_OK) return s;
    }
  }
  ~DescLease() { if (idx >= 0 && p->descs[idx].busy == kLeased) p->descs[idx].busy = 0; }
};

// drop the references blocks[from, to) of a request, in logical order; freed ids join the tail
void unref(kvr_pool *p, const Request &r, int32_t from, int32_t to) {
  for (int32_t i = from; i < to; ++i) p->fq.drop_ref(r.blocks[i]);
}

// a request lets go of every block it refers to (its whole table, or the kept prefix while on the host)
void drop_all_blocks(kvr_pool *p, Request &r) {
  unref(p, r, 0, (int32_t)r.blocks.size());
  std::vector<int32_t>().swap(r.blocks);
}

void free_host(kvr_pool *p, Request &r, uint64_t reader_seq) {
  if (r.arena_len) {
    p->arena.release(r.arena_off, r.arena_len);
    if (reader_seq) p->pending_free.push_back({r.arena_off, r.arena_len, reader_seq});
  }
  r.arena_off = r.arena_len = 0;
}

inline int64_t private_tokens(const kvr_pool *p, const Request &r) { return r.n_tokens - (int64_t)r.n_shared * p->BS; }

// shared body of the four bookkeeping-only outcomes and of the per-request loops
struct Batch {
  kvr_status acc = KVR_OK;
  kvr_status *per;
  int i = 0;
  void put(kvr_status s) { if (per) per[i] = s; acc = fold(acc, s); ++i; }
};

// Who may donate its first n_shared blocks as a shared prefix: a request that still refers to them -- ACTIVE or
// RETAINED with that many full blocks, or on the HOST with a kept prefix at least that long.
kvr_status check_donor(kvr_pool *p, uint64_t id, uint64_t donor_id, int32_t n_shared, const Request **out) {
  if (donor_id == id) return fail(KVR_ERR_INVALID_ARG, "a request cannot share with itself");
  auto d = p->reqs.find(donor_id);
  if (d == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown donor");
  const Request &donor = d->second;
  if (donor.state == KVR_ACTIVE || donor.state == KVR_RETAINED) {
    if ((int64_t)n_shared * p->BS > donor.n_tokens) return fail(KVR_ERR_INVALID_ARG, "the donor has fewer full blocks");
  } else if (donor.state == KVR_HOST) {
    if (n_shared > donor.n_shared) return fail(KVR_ERR_INVALID_ARG, "a donor on the host refers only to its own shared prefix");
  } else {
    return fail(KVR_ERR_BAD_STATE, "a discarded donor refers to no blocks");
  }
  *out = &donor;
  return KVR_OK;
}

// the new request's table: donor prefix (one more reference each) followed by ids from the head of the queue
kvr_status admit_common(kvr_pool *p, std::unique_lock<std::mutex> &lock, uint64_t id, int64_t n_tokens, const Request *donor,
                        int32_t n_shared, int32_t *out_blocks) {
  const int64_t nb = (n_tokens + p->BS - 1) / p->BS;
  if (nb - n_shared > p->fq.size()) { p->st.hbm_full_rejects++; return KVR_HBM_FULL; }
  std::vector<int32_t> table((size_t)nb);
  for (int32_t i = 0; i < n_shared; ++i) table[i] = donor->blocks[i];
  Request &r = p->reqs[id];                        // may rehash: `donor` is not used below
  r = Request();
  r.state = KVR_ACTIVE; r.n_tokens = n_tokens; r.nb = (int32_t)nb; r.n_shared = n_shared;
  r.image_bytes = (uint64_t)(n_tokens - (int64_t)n_shared * p->BS) * p->bpt;
  r.blocks.swap(table);
  for (int32_t i = 0; i < n_shared; ++i) p->fq.add_ref(r.blocks[i]);
  const uint64_t tag = p->fq.pop((int32_t)nb - n_shared, r.blocks.data() + n_shared);
  if (out_blocks && nb) memcpy(out_blocks, r.blocks.data(), (size_t)nb * 4);
  // the caller will write the new blocks from its own stream: let any gather still reading them finish
  if (tag && !p->meta_only) return wait_unlocked(p, lock, tag, true, 60000);
  return KVR_OK;
}

}  // namespace

// ---- C ABI -------------------------------------------------------------------------------

extern "C" {

const char *kvr_last_error(void) { return last_error_text(); }

uint64_t kvr_bytes_per_token(const kvr_geometry *g) {
  if (!g || g->layers < 1 || g->kv_heads < 1 || g->head_dim < 1 || g->block_size < 1) return 0;
  if (g->dtype_bytes != 1 && g->dtype_bytes != 2 && g->dtype_bytes != 4) return 0;
  const uint64_t row = (uint64_t)g->kv_heads * g->head_dim * g->dtype_bytes;
  if (row % 16) return 0;
  return 2ull * g->layers * row;
}

kvr_status kvr_pool_create(const kvr_config *cfg, kvr_pool **out) {
  if (!cfg || !out) return fail(KVR_ERR_INVALID_ARG, "cfg or out is NULL");
  const uint64_t bpt = kvr_bytes_per_token(&cfg->g);
  if (!bpt) return fail(KVR_ERR_GEOMETRY, "invalid geometry (fields >= 1, dtype_bytes in {1,2,4}, row bytes multiple of 16)");
  if (cfg->num_blocks < 1) return fail(KVR_ERR_INVALID_ARG, "num_blocks < 1");
  const uint64_t row = bpt / 2 / cfg->g.layers, tile = row * cfg->g.block_size;
  if (tile > (1u << 30)) return fail(KVR_ERR_GEOMETRY, "one tile exceeds 1 GiB");
  kvr_pool *p = new (std::nothrow) kvr_pool();
  if (!p) return fail(KVR_ERR_NOMEM, "out of host memory");
  p->cfg = *cfg;
  if (!p->cfg.chunk_bytes) {
    p->cfg.chunk_bytes = 64ull << 20;
    if (p->cfg.chunk_bytes < tile) p->cfg.chunk_bytes = align_up(tile, 4096);
  }
  if (!p->cfg.staging_slots) p->cfg.staging_slots = 32;
  if (!p->cfg.kernel) p->cfg.kernel = KVR_KERNEL_BULK;
  if (!p->cfg.max_moves_in_flight) p->cfg.max_moves_in_flight = 16;
  if (p->cfg.suspend_single_bytes) p->suspend_single = p->cfg.suspend_single_bytes;
  if (p->cfg.resume_single_bytes) p->resume_single = p->cfg.resume_single_bytes;
  if (p->cfg.copy_piece_bytes) p->copy_piece = p->cfg.copy_piece_bytes;
  kvr_status bad = KVR_OK;
  if (p->cfg.route < KVR_ROUTE_AUTO || p->cfg.route > KVR_ROUTE_DMA2D) bad = fail(KVR_ERR_INVALID_ARG, "unknown route");
  else if (p->cfg.layout != KVR_LAYER_MAJOR && p->cfg.layout != KVR_BLOCK_MAJOR) bad = fail(KVR_ERR_INVALID_ARG, "unknown layout");
  else if (p->cfg.kernel != KVR_KERNEL_WARP && p->cfg.kernel != KVR_KERNEL_BULK) bad = fail(KVR_ERR_INVALID_ARG, "unknown kernel");
  else if (p->cfg.chunk_bytes % 4096 || p->cfg.chunk_bytes < tile) bad = fail(KVR_ERR_INVALID_ARG, "chunk_bytes must be a multiple of 4096 and hold one tile");
  else if (p->cfg.staging_slots < 2 || p->cfg.staging_slots > 64) bad = fail(KVR_ERR_INVALID_ARG, "staging_slots must be in [2, 64]");
  else if (p->cfg.max_ctas < 0) bad = fail(KVR_ERR_INVALID_ARG, "max_ctas < 0");
  else if (p->cfg.max_moves_in_flight < 1 || p->cfg.max_moves_in_flight > 256) bad = fail(KVR_ERR_INVALID_ARG, "max_moves_in_flight must be in [1, 256]");
  else if (p->copy_piece < 4096 || p->copy_piece % 4096) bad = fail(KVR_ERR_INVALID_ARG, "copy_piece_bytes must be a multiple of 4096");
  if (!bad && cfg->initial_free_order) {
    std::vector<uint8_t> seen(cfg->num_blocks, 0);
    for (int32_t i = 0; i < cfg->num_blocks && !bad; ++i) {
      const int32_t b = cfg->initial_free_order[i];
      if (b < 0 || b >= cfg->num_blocks || seen[b]) bad = fail(KVR_ERR_INVALID_ARG, "initial_free_order is not a permutation");
      else seen[b] = 1;
    }
  }
  if (bad) { delete p; return bad; }
  p->meta_only = cfg->flags & KVR_METADATA_ONLY;
  p->profile = cfg->flags & KVR_PROFILE;
  p->bpt = bpt; p->row = (int)row; p->tile_bytes = (int)tile;
  p->NB = cfg->num_blocks; p->BS = cfg->g.block_size; p->planes = 2 * cfg->g.layers;
  if (p->cfg.layout == KVR_BLOCK_MAJOR) { p->plane_stride = p->tile_bytes; p->block_stride = (long long)p->planes * p->tile_bytes; }
  else { p->plane_stride = (long long)p->NB * p->tile_bytes; p->block_stride = p->tile_bytes; }
  p->fq.init(p->NB, cfg->initial_free_order);
  p->arena.init(cfg->host_capacity_bytes);
  p->cfg.initial_free_order = nullptr;
  if (!p->meta_only) {
    kvr_status s = create_engine(p);
    if (s != KVR_OK) { destroy_engine(p); delete p; return s; }
  }
  *out = p;
  return KVR_OK;
}

kvr_status kvr_pool_destroy(kvr_pool *p) {
  if (!p) return KVR_OK;
  kvr_status s = KVR_OK;
  if (!p->meta_only) {
    cudaSetDevice(p->device);
    s = wait_locked(p, 0, 60000);
    if (s != KVR_OK) cudaDeviceSynchronize();
    destroy_engine(p);
  }
  delete p;
  return s;
}

kvr_status kvr_request_admit(kvr_pool *p, uint64_t id, int64_t n_tokens, int32_t *out_blocks, int32_t cap) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n_tokens < 0) return fail(KVR_ERR_INVALID_ARG, "n_tokens < 0");
  const int64_t nb = (n_tokens + p->BS - 1) / p->BS;
  if (out_blocks && cap < nb) return fail(KVR_ERR_INVALID_ARG, "out_blocks too small");
  auto it = p->reqs.find(id);
  if (it != p->reqs.end() && it->second.state != KVR_EXPIRED) return fail(KVR_ERR_BAD_STATE, "request exists");
  try {
    return admit_common(p, enter.lock, id, n_tokens, nullptr, 0, out_blocks);
  } catch (const std::bad_alloc &) {
    return fail(KVR_ERR_NOMEM, "out of host memory");
  }
}

kvr_status kvr_request_admit_sharing(kvr_pool *p, uint64_t id, int64_t n_tokens, uint64_t donor_id, int32_t n_shared,
                                     int32_t *out_blocks, int32_t cap) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n_tokens < 0 || n_shared < 0) return fail(KVR_ERR_INVALID_ARG, "negative size");
  const int64_t nb = (n_tokens + p->BS - 1) / p->BS;
  if ((int64_t)n_shared * p->BS > n_tokens) return fail(KVR_ERR_INVALID_ARG, "the shared prefix must be whole blocks inside the request");
  if (out_blocks && cap < nb) return fail(KVR_ERR_INVALID_ARG, "out_blocks too small");
  auto it = p->reqs.find(id);
  if (it != p->reqs.end() && it->second.state != KVR_EXPIRED) return fail(KVR_ERR_BAD_STATE, "request exists");
  const Request *donor = nullptr;
  if (n_shared > 0) { if (kvr_status s = check_donor(p, id, donor_id, n_shared, &donor)) return s; }
  try {
    return admit_common(p, enter.lock, id, n_tokens, donor, n_shared, out_blocks);
  } catch (const std::bad_alloc &) {
    return fail(KVR_ERR_NOMEM, "out of host memory");
  }
}

kvr_status kvr_request_admit_sharing_into(kvr_pool *p, uint64_t id, int64_t n_tokens, uint64_t donor_id, int32_t n_shared,
                                          const int32_t *private_blocks, int32_t n_private) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n_tokens < 0 || n_shared < 0 || n_private < 0 || (n_private > 0 && !private_blocks)) return fail(KVR_ERR_INVALID_ARG, "bad size or block list");
  if ((int64_t)n_shared * p->BS > n_tokens) return fail(KVR_ERR_INVALID_ARG, "the shared prefix must be whole blocks inside the request");
  if ((n_tokens + p->BS - 1) / p->BS != (int64_t)n_shared + (int64_t)n_private)
    return fail(KVR_ERR_INVALID_ARG, "shared + private blocks must equal ceil(n_tokens / block_size)");
  auto it = p->reqs.find(id);
  if (it != p->reqs.end() && it->second.state != KVR_EXPIRED) return fail(KVR_ERR_BAD_STATE, "request exists");
  const bool existed = it != p->reqs.end();
  try {
    const int32_t nb = n_shared + n_private;
    std::vector<int32_t> table((size_t)nb), prevs((size_t)n_private);
    if (n_shared > 0) {
      const Request *donor = nullptr;
      if (kvr_status s = check_donor(p, id, donor_id, n_shared, &donor)) return s;
      for (int32_t i = 0; i < n_shared; ++i) table[i] = donor->blocks[i];
    }
    Request &r = p->reqs[id];
    uint64_t tag = 0;
    int32_t bad = -1;
    if (!p->fq.claim(private_blocks, n_private, prevs.data(), &tag, &bad)) {
      if (!existed) p->reqs.erase(id);
      return fail(KVR_ERR_INVALID_ARG, "block %d is not free or named twice", bad);
    }
    for (int32_t i = 0; i < n_private; ++i) table[n_shared + i] = private_blocks[i];
    r = Request();
    r.state = KVR_ACTIVE; r.n_tokens = n_tokens; r.nb = nb; r.n_shared = n_shared;
    r.image_bytes = (uint64_t)(n_tokens - (int64_t)n_shared * p->BS) * p->bpt;
    r.blocks.swap(table);
    for (int32_t i = 0; i < n_shared; ++i) p->fq.add_ref(r.blocks[i]);
    if (tag && !p->meta_only) return wait_unlocked(p, enter.lock, tag, true, 60000);     // a gather may still be reading the named blocks
    return KVR_OK;
  } catch (const std::bad_alloc &) {
    return fail(KVR_ERR_NOMEM, "out of host memory");
  }
}

kvr_status kvr_request_admit_into(kvr_pool *p, uint64_t id, int64_t n_tokens, const int32_t *blocks, int32_t nb) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n_tokens < 0 || nb < 0 || (nb > 0 && !blocks)) return fail(KVR_ERR_INVALID_ARG, "bad size or block list");
  if ((n_tokens + p->BS - 1) / p->BS != (int64_t)nb) return fail(KVR_ERR_INVALID_ARG, "nb must equal ceil(n_tokens / block_size)");
  auto it = p->reqs.find(id);
  if (it != p->reqs.end() && it->second.state != KVR_EXPIRED) return fail(KVR_ERR_BAD_STATE, "request exists");
  const bool existed = it != p->reqs.end();
  try {
    std::vector<int32_t> table(blocks, blocks + nb), prevs((size_t)nb);
    Request &r = p->reqs[id];
    uint64_t tag = 0;
    int32_t bad = -1;
    if (!p->fq.claim(blocks, nb, prevs.data(), &tag, &bad)) {
      if (!existed) p->reqs.erase(id);
      return fail(KVR_ERR_INVALID_ARG, "block %d is not free or named twice", bad);
    }
    r = Request();
    r.state = KVR_ACTIVE; r.n_tokens = n_tokens; r.nb = nb;
    r.image_bytes = (uint64_t)n_tokens * p->bpt;
    r.blocks.swap(table);
    if (tag && !p->meta_only) return wait_unlocked(p, enter.lock, tag, true, 60000);     // a gather may still be reading these blocks
    return KVR_OK;
  } catch (const std::bad_alloc &) {
    return fail(KVR_ERR_NOMEM, "out of host memory");
  }
}

kvr_status kvr_request_release(kvr_pool *p, uint64_t id) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  for (;;) {
    auto it = p->reqs.find(id);
    if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
    Request &r = it->second;
    if (r.pending_op) {            // the request must be at rest; the lock is given up meanwhile, so look again after
      if (kvr_status s = wait_unlocked(p, enter.lock, r.pending_op, false, 60000)) return s;
      continue;
    }
    if (r.state == KVR_HOST) free_host(p, r, 0);
    if (r.state != KVR_EXPIRED) drop_all_blocks(p, r);
    p->reqs.erase(it);
    return KVR_OK;
  }
}

kvr_status kvr_retain_in_hbm(kvr_pool *p, const uint64_t *req, int32_t n, kvr_status *per_req) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n < 0 || (n > 0 && !req)) return fail(KVR_ERR_INVALID_ARG, "bad request list");
  Batch b{KVR_OK, per_req};
  for (int32_t i = 0; i < n; ++i) {
    auto it = p->reqs.find(req[i]);
    if (it == p->reqs.end()) { b.put(KVR_ERR_UNKNOWN_REQUEST); continue; }
    if (it->second.state != KVR_ACTIVE) { b.put(KVR_ERR_BAD_STATE); continue; }
    it->second.state = KVR_RETAINED;
    b.put(KVR_OK);
  }
  return b.acc;
}

kvr_status kvr_expire(kvr_pool *p, const uint64_t *req, int32_t n, kvr_status *per_req) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n < 0 || (n > 0 && !req)) return fail(KVR_ERR_INVALID_ARG, "bad request list");
  Batch b{KVR_OK, per_req};
  for (int32_t i = 0; i < n; ++i) {
    for (;;) {
      auto it = p->reqs.find(req[i]);
      if (it == p->reqs.end()) { b.put(KVR_ERR_UNKNOWN_REQUEST); break; }
      Request &r = it->second;
      if (r.state == KVR_EXPIRED) { b.put(KVR_ERR_BAD_STATE); break; }
      if (r.pending_op) {          // settle the move in flight first (lock given up meanwhile: look again after)
        if (kvr_status s = wait_unlocked(p, enter.lock, r.pending_op, false, 60000)) { b.put(s); break; }
        continue;
      }
      if (r.state == KVR_HOST) { p->st.bytes_expired_from_host += r.image_bytes; free_host(p, r, 0); }
      drop_all_blocks(p, r);
      r.state = KVR_EXPIRED;
      p->st.expires++; p->st.recompute_marked++;
      b.put(KVR_OK);
      break;
    }
  }
  return b.acc;
}

kvr_status kvr_suspend_to_host(kvr_pool *p, const uint64_t *req, int32_t n, uint32_t flags, kvr_status *per_req) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n < 0 || (n > 0 && !req)) return fail(KVR_ERR_INVALID_ARG, "bad request list");
  const auto t_call = Clock::now();
  DescLease lease(p);
  if (kvr_status s = lease.take(enter.lock)) return s;
  Batch b{KVR_OK, per_req};
  std::vector<Item> items;
  std::vector<uint64_t> arena_waits;
  uint64_t seq = 0;
  int64_t rejects = 0;
  kvr_status err = KVR_OK;
  try {
    alloc_point(p);
    items.reserve((size_t)n);
    alloc_point(p);
    p->pending_free.reserve(p->pending_free.size() + (size_t)n);
    for (int32_t i = 0; i < n; ++i) {
      auto it = p->reqs.find(req[i]);
      if (it == p->reqs.end()) { b.put(KVR_ERR_UNKNOWN_REQUEST); continue; }
      Request &r = it->second;
      if (r.state != KVR_ACTIVE && r.state != KVR_RETAINED) { b.put(KVR_ERR_BAD_STATE); continue; }
      const uint64_t len = align_up(r.image_bytes, kArenaGranule);
      uint64_t off = 0;
      if (len && !p->arena.alloc(len, &off)) { p->st.host_full_rejects++; ++rejects; b.put(KVR_HOST_FULL); continue; }
      r.arena_off = off; r.arena_len = len;
      // only the private suffix moves: the part of the table behind the shared prefix
      items.push_back({req[i], &r, r.blocks.data() + r.n_shared, r.nb - r.n_shared, private_tokens(p, r), off, 0, i, r.state});
      r.state = KVR_HOST;
      p->st.suspends++; p->st.bytes_suspended += r.image_bytes;
      b.put(KVR_OK);
    }
    if (!p->meta_only && !items.empty()) {
      for (auto &it : items)
        for (auto &pf : p->pending_free)
          if (it.r->arena_len && pf.off < it.r->arena_off + it.r->arena_len && it.r->arena_off < pf.off + pf.len) {
            alloc_point(p);
            arena_waits.push_back(pf.seq);
          }
      err = enqueue(p, OP_SUSPEND, items, p->route, nullptr, 0, arena_waits, t_call, lease.idx, &seq);
    }
  } catch (const std::bad_alloc &) {
    err = fail(KVR_ERR_NOMEM, "out of host memory");
  }
  if (err != KVR_OK) {
    // nothing was moved: every request of the batch goes back to exactly what it was
    for (size_t k = items.size(); k-- > 0;) {
      Request &r = *items[k].r;
      if (r.arena_len) p->arena.release(r.arena_off, r.arena_len);
      r.arena_off = r.arena_len = 0;
      r.state = items[k].prev_state;
      p->st.suspends--; p->st.bytes_suspended -= r.image_bytes;
      if (per_req) per_req[items[k].batch_index] = err;
    }
    p->st.host_full_rejects -= rejects;      // a rejection seen only because earlier requests of this batch held room
    return fold(b.acc, err);
  }
  // the move has copied the tables; now the private ids are let go in request order, each in logical block order
  // (a block joins the free tail when its last reference goes), remembered as read by this move
  for (auto &it : items) {
    Request &r = *it.r;
    p->fq.note_reader(it.blocks, it.nb, seq);
    unref(p, r, r.n_shared, r.nb);
    if (r.n_shared) r.blocks.resize(r.n_shared); else std::vector<int32_t>().swap(r.blocks);
  }
  if (seq && (flags & KVR_SYNC)) { if (kvr_status s = wait_unlocked(p, enter.lock, seq, false, 60000)) return s; }
  return b.acc;
}

// what a resume took and must give back if the move cannot be enqueued
struct Taken { bool named = false; std::vector<int32_t> prevs; };

static kvr_status resume_commit_or_rollback(kvr_pool *p, std::unique_lock<std::mutex> &lock, std::vector<Item> &items,
                                            std::vector<Taken> &taken, uint64_t block_tag, uint32_t flags,
                                            Clock::time_point t_call, int lease, kvr_status err, kvr_status *per_req,
                                            bool *rolled_back) {
  uint64_t seq = 0;
  *rolled_back = false;
  if (err == KVR_OK && !p->meta_only && !items.empty()) {
    try {
      std::vector<uint64_t> none;
      p->call_flags = flags;
      err = enqueue(p, OP_RESUME, items, p->route, nullptr, block_tag, none, t_call, lease, &seq);
    } catch (const std::bad_alloc &) {
      err = fail(KVR_ERR_NOMEM, "out of host memory");
    }
    p->call_flags = 0;
  }
  if (err != KVR_OK) {
    // nothing was moved: the blocks go back where they came from (last taken first), the images stay on the host
    for (size_t k = items.size(); k-- > 0;) {
      Request &r = *items[k].r;
      int32_t *mine = r.blocks.data() + r.n_shared;
      if (taken[k].named) p->fq.unclaim(mine, taken[k].prevs.data(), r.nb - r.n_shared);
      else p->fq.unpop(mine, r.nb - r.n_shared);
      r.blocks.resize(r.n_shared);
      r.state = KVR_HOST;
      p->st.resumes--; p->st.bytes_resumed -= r.image_bytes;
      if (per_req) per_req[items[k].batch_index] = err;
    }
    *rolled_back = true;
    return err;
  }
  for (auto &it : items) free_host(p, *it.r, seq);
  if (seq && (flags & KVR_SYNC)) return wait_unlocked(p, lock, seq, false, 60000);
  return KVR_OK;
}

kvr_status kvr_resume_from_host(kvr_pool *p, const uint64_t *req, int32_t n, uint32_t flags, kvr_status *per_req) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n < 0 || (n > 0 && !req)) return fail(KVR_ERR_INVALID_ARG, "bad request list");
  const auto t_call = Clock::now();
  DescLease lease(p);
  if (kvr_status s = lease.take(enter.lock)) return s;
  Batch b{KVR_OK, per_req};
  std::vector<Item> items;
  std::vector<Taken> taken;
  uint64_t block_tag = 0;
  int64_t rejects = 0;
  kvr_status err = KVR_OK;
  try {
    alloc_point(p);
    items.reserve((size_t)n);
    taken.resize((size_t)n);
    alloc_point(p);
    p->pending_free.reserve(p->pending_free.size() + (size_t)n);
    for (int32_t i = 0; i < n; ++i) {
      auto it = p->reqs.find(req[i]);
      if (it == p->reqs.end()) { b.put(KVR_ERR_UNKNOWN_REQUEST); continue; }
      Request &r = it->second;
      if (r.state == KVR_RETAINED) { r.state = KVR_ACTIVE; p->st.resident_resumes++; b.put(KVR_RESIDENT); continue; }
      if (r.state == KVR_EXPIRED) { b.put(KVR_RECOMPUTE); continue; }
      if (r.state != KVR_HOST) { b.put(KVR_ERR_BAD_STATE); continue; }
      const int32_t n_priv = r.nb - r.n_shared;
      if (n_priv > p->fq.size()) { p->st.hbm_full_rejects++; ++rejects; b.put(KVR_HBM_FULL); continue; }
      alloc_point(p);
      r.blocks.resize(r.nb);                       // the kept prefix, then the fresh private blocks
      const uint64_t tag = p->fq.pop(n_priv, r.blocks.data() + r.n_shared);
      if (tag > block_tag) block_tag = tag;
      items.push_back({req[i], &r, nullptr, n_priv, private_tokens(p, r), r.arena_off, 0, i, KVR_HOST});
      r.state = KVR_ACTIVE;
      p->st.resumes++; p->st.bytes_resumed += r.image_bytes;
      b.put(KVR_OK);
    }
    for (auto &it : items) it.blocks = it.r->blocks.data() + it.r->n_shared;
  } catch (const std::bad_alloc &) {
    err = fail(KVR_ERR_NOMEM, "out of host memory");
    for (auto &it : items) it.blocks = it.r->blocks.data() + it.r->n_shared;
  }
  taken.resize(items.size());
  bool rolled_back = false;
  if (kvr_status s = resume_commit_or_rollback(p, enter.lock, items, taken, block_tag, flags, t_call, lease.idx, err, per_req, &rolled_back)) {
    if (rolled_back) p->st.hbm_full_rejects -= rejects;    // a rejection seen only because earlier requests of this batch took blocks
    return fold(b.acc, s);
  }
  return b.acc;
}

kvr_status kvr_resume_from_host_into(kvr_pool *p, uint64_t req, const int32_t *blocks, int32_t nb, uint32_t flags) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (nb < 0 || (nb > 0 && !blocks)) return fail(KVR_ERR_INVALID_ARG, "bad block list");
  const auto t_call = Clock::now();
  DescLease lease(p);
  if (kvr_status s = lease.take(enter.lock)) return s;
  auto it = p->reqs.find(req);
  if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
  Request &r = it->second;
  if (r.state != KVR_HOST) return fail(KVR_ERR_BAD_STATE, "request is not on the host");
  if (nb != r.nb - r.n_shared) return fail(KVR_ERR_INVALID_ARG, "request has %d private blocks, %d named", r.nb - r.n_shared, nb);
  std::vector<Item> items;
  std::vector<Taken> taken(1);
  uint64_t tag = 0;
  try {
    alloc_point(p);
    items.reserve(1);
    taken[0].named = true;
    taken[0].prevs.resize((size_t)nb);
    alloc_point(p);
    p->pending_free.reserve(p->pending_free.size() + 1);
    alloc_point(p);
    r.blocks.reserve((size_t)r.nb);
  } catch (const std::bad_alloc &) {
    return fail(KVR_ERR_NOMEM, "out of host memory");
  }
  int32_t bad = -1;
  if (!p->fq.claim(blocks, nb, taken[0].prevs.data(), &tag, &bad)) return fail(KVR_ERR_INVALID_ARG, "block %d is not free or named twice", bad);
  r.blocks.insert(r.blocks.end(), blocks, blocks + nb);          // capacity reserved above
  items.push_back({req, &r, r.blocks.data() + r.n_shared, nb, private_tokens(p, r), r.arena_off, 0, 0, KVR_HOST});
  r.state = KVR_ACTIVE;
  p->st.resumes++; p->st.bytes_resumed += r.image_bytes;
  bool rolled_back = false;
  return resume_commit_or_rollback(p, enter.lock, items, taken, tag, flags, t_call, lease.idx, KVR_OK, nullptr, &rolled_back);
}

static kvr_status device_copy(kvr_pool *p, int kind, const uint64_t *req, int32_t n, char *dev, uint64_t capacity,
                              uint64_t *offsets, uint32_t flags) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (p->meta_only) return fail(KVR_ERR_BAD_STATE, "metadata-only pool moves no data");
  if (n < 0 || (n > 0 && !req) || !dev || ((uintptr_t)dev & 255)) return fail(KVR_ERR_INVALID_ARG, "bad request list or buffer (256-byte aligned device pointer)");
  const auto t_call = Clock::now();
  DescLease lease(p);
  if (kvr_status s = lease.take(enter.lock)) return s;
  try {
    std::vector<Item> items;
    uint64_t cursor = 0;
    for (int32_t i = 0; i < n; ++i) {
      auto it = p->reqs.find(req[i]);
      if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
      Request &r = it->second;
      if (r.state != KVR_ACTIVE && r.state != KVR_RETAINED) return fail(KVR_ERR_BAD_STATE, "request holds no blocks");
      cursor = align_up(cursor, 256);
      if (offsets) offsets[i] = cursor;
      items.push_back({req[i], &r, r.blocks.data(), r.nb, r.n_tokens, cursor, 0, i, r.state});   // the whole request, shared prefix included
      cursor += (uint64_t)r.n_tokens * p->bpt;
    }
    if (cursor > capacity) return fail(KVR_ERR_INVALID_ARG, "buffer holds %llu bytes, %llu needed", (unsigned long long)capacity, (unsigned long long)cursor);
    uint64_t seq = 0;
    std::vector<uint64_t> none;
    if (!items.empty())
      if (kvr_status s = enqueue(p, kind, items, 0, dev, 0, none, t_call, lease.idx, &seq)) return s;
    if (seq && (flags & KVR_SYNC)) return wait_unlocked(p, enter.lock, seq, false, 60000);
    return KVR_OK;
  } catch (const std::bad_alloc &) {
    return fail(KVR_ERR_NOMEM, "out of host memory");
  }
}

kvr_status kvr_export_to_device(kvr_pool *p, const uint64_t *req, int32_t n, void *dst, uint64_t capacity,
                                uint64_t *offsets, uint32_t flags) {
  return device_copy(p, OP_EXPORT, req, n, (char *)dst, capacity, offsets, flags);
}

kvr_status kvr_import_from_device(kvr_pool *p, const uint64_t *req, int32_t n, const void *src, uint64_t capacity,
                                  uint64_t *offsets, uint32_t flags) {
  return device_copy(p, OP_IMPORT, req, n, (char *)src, capacity, offsets, flags);
}

kvr_status kvr_request_info(kvr_pool *p, uint64_t req, int32_t *state, int64_t *n_tokens, int32_t *nb, int32_t *blocks,
                            int32_t cap, const void **host_image, uint64_t *image_bytes, uint64_t *arena_offset) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (!p->meta_only) { if (kvr_status s = poll(p)) return s; }
  auto it = p->reqs.find(req);
  if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
  const Request &r = it->second;
  const bool held = r.state == KVR_ACTIVE || r.state == KVR_RETAINED;
  if (state) {
    // a move in flight shows as SUSPENDING / RESUMING until it lands, unless a later call has already moved the
    // settled state on (a resuming request that was retained again reports RETAINED)
    const bool transient = r.pending_op && ((r.pending_kind == KVR_SUSPENDING && r.state == KVR_HOST) ||
                                            (r.pending_kind == KVR_RESUMING && r.state == KVR_ACTIVE));
    *state = transient ? r.pending_kind : r.state;
  }
  if (n_tokens) *n_tokens = r.n_tokens;
  if (nb) *nb = r.nb;
  if (blocks && held) {
    if (cap < r.nb) return fail(KVR_ERR_INVALID_ARG, "blocks too small");
    if (r.nb) memcpy(blocks, r.blocks.data(), (size_t)r.nb * 4);
  }
  if (host_image) *host_image = (r.state == KVR_HOST && p->h_arena) ? p->h_arena + r.arena_off : nullptr;
  if (image_bytes) *image_bytes = r.image_bytes;
  if (arena_offset) *arena_offset = r.state == KVR_HOST ? r.arena_off : 0;
  return KVR_OK;
}

kvr_status kvr_request_sharing(kvr_pool *p, uint64_t req, int32_t *n_shared, int32_t *blocks, int32_t cap) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  auto it = p->reqs.find(req);
  if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
  const Request &r = it->second;
  const int32_t ns = r.state == KVR_EXPIRED ? 0 : r.n_shared;
  if (n_shared) *n_shared = ns;
  if (blocks) {
    if (cap < ns) return fail(KVR_ERR_INVALID_ARG, "blocks too small");
    if (ns) memcpy(blocks, r.blocks.data(), (size_t)ns * 4);
  }
  return KVR_OK;
}

int32_t kvr_block_refcount(kvr_pool *p, int32_t block) {
  if (!p) return -1;
  Enter enter(p);
  if (block < 0 || block >= p->NB) return -1;
  return p->fq.refs(block);
}

kvr_status kvr_request_latency(kvr_pool *p, uint64_t req, double *host_ms, double *device_ms) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (!p->meta_only) { if (kvr_status s = poll(p)) return s; }
  auto it = p->reqs.find(req);
  if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
  if (it->second.pending_op || !it->second.has_latency) return fail(KVR_ERR_BAD_STATE, "no completed move to report");
  if (host_ms) *host_ms = it->second.host_ms;
  if (device_ms) *device_ms = it->second.device_ms;
  return KVR_OK;
}

kvr_status kvr_wait(kvr_pool *p, uint64_t req_or_all, int64_t timeout_ms) {
  if (kvr_status s = check_pool(p)) return s;
  if (p->meta_only) return KVR_OK;
  Enter enter(p);
  uint64_t seq = 0;
  if (req_or_all != KVR_ALL) {
    auto it = p->reqs.find(req_or_all);
    if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
    seq = it->second.pending_op;
    if (!seq) return KVR_OK;
  }
  // the lock is held per look, not while sleeping, so other threads keep working on the pool meanwhile
  return wait_unlocked(p, enter.lock, seq, false, timeout_ms);
}

kvr_status kvr_pool_stats(kvr_pool *p, kvr_stats *out) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (!out) return fail(KVR_ERR_INVALID_ARG, "out is NULL");
  if (!p->meta_only) { if (kvr_status s = poll(p)) return s; }
  kvr_stats s = p->st;
  s.blocks_total = p->NB; s.blocks_free = p->fq.size();
  s.blocks_active = s.blocks_pinned = 0;
  s.n_active = s.n_retained = s.n_host = s.n_expired = 0;
  // distinct blocks: 1 = held by active requests only, 2 = named by a suspended context (retained, or the prefix a
  // request on the host still refers to)
  std::vector<uint8_t> mark;
  try { mark.assign((size_t)p->NB, 0); } catch (const std::bad_alloc &) { return fail(KVR_ERR_NOMEM, "out of host memory"); }
  for (auto &kv : p->reqs) {
    const Request &r = kv.second;
    if (r.state == KVR_ACTIVE) s.n_active++;
    else if (r.state == KVR_RETAINED) s.n_retained++;
    else if (r.state == KVR_HOST) s.n_host++;
    else if (r.state == KVR_EXPIRED) s.n_expired++;
    const uint8_t m = r.state == KVR_ACTIVE ? 1 : 2;
    for (int32_t b : r.blocks) if (mark[b] < m) mark[b] = m;
  }
  for (uint8_t m : mark) { if (m == 1) s.blocks_active++; else if (m == 2) s.blocks_pinned++; }
  s.host_capacity = p->arena.capacity(); s.host_used = p->arena.used(); s.host_largest_hole = p->arena.largest_hole();
  s.ops_in_flight = (int64_t)p->ops.size();
  *out = s;
  return KVR_OK;
}

int64_t kvr_free_queue(kvr_pool *p, int32_t *out, int64_t cap) {
  if (!p) return -1;
  Enter enter(p);
  const int64_t n = p->fq.size();
  if (out) {
    int64_t i = 0;
    for (int32_t b = p->fq.first(); b >= 0 && i < cap; b = p->fq.after(b)) out[i++] = b;
  }
  return n;
}

kvr_status kvr_test_fail_nth(kvr_pool *p, int32_t kind, int64_t n) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if ((kind != KVR_FAIL_CUDA && kind != KVR_FAIL_ALLOC) || n < 0) return fail(KVR_ERR_INVALID_ARG, "kind is KVR_FAIL_CUDA or KVR_FAIL_ALLOC, n >= 0");
  p->inject[kind] = n;
  p->points[kind] = 0;
  return KVR_OK;
}

int64_t kvr_test_points(kvr_pool *p, int32_t kind) {
  if (!p || (kind != KVR_FAIL_CUDA && kind != KVR_FAIL_ALLOC)) return -1;
  Enter enter(p);
  return p->points[kind];
}

kvr_status kvr_test_plan(const kvr_geometry *g, const int64_t *n_tokens, int32_t n_items, uint64_t slot_bytes, int32_t slots,
                         int32_t launch_slots, int32_t ring_next, int32_t resume, uint32_t flags, uint64_t suspend_single,
                         uint64_t resume_single, int64_t *chunks, int64_t *copies, int64_t *segs, int64_t cap, int64_t *counts) {
  const uint64_t bpt = kvr_bytes_per_token(g);
  if (!bpt || !n_tokens || n_items < 0 || slots < 2 || launch_slots < 1 || launch_slots >= slots || ring_next < 0 ||
      ring_next >= slots || !chunks || !copies || !segs || !counts || cap < 0)
    return fail(KVR_ERR_INVALID_ARG, "kvr_test_plan: bad arguments");
  try {
    kvr_pool pool;                                  // bookkeeping fields only: the planner touches nothing else
    kvr_pool *p = &pool;
    p->bpt = bpt; p->row = (int)(bpt / 2 / g->layers); p->tile_bytes = p->row * g->block_size;
    p->BS = g->block_size; p->planes = 2 * g->layers;
    if (slot_bytes % 4096 || slot_bytes < (uint64_t)p->tile_bytes) return fail(KVR_ERR_INVALID_ARG, "kvr_test_plan: slot size");
    p->slot_bytes = slot_bytes; p->launch_slots = launch_slots; p->call_flags = flags;
    if (suspend_single) p->suspend_single = suspend_single;
    if (resume_single) p->resume_single = resume_single;
    Ring ring;
    ring.base = reinterpret_cast<char *>(uintptr_t(1) << 40);   // never dereferenced
    ring.slots.resize((size_t)slots);
    ring.next = ring_next;
    std::vector<Item> items;
    uint64_t lin = 0, bt = 0;
    for (int32_t i = 0; i < n_items; ++i) {
      if (n_tokens[i] < 0) return fail(KVR_ERR_INVALID_ARG, "kvr_test_plan: negative length");
      const int32_t nb = (int32_t)((n_tokens[i] + p->BS - 1) / p->BS);
      items.push_back({(uint64_t)i, nullptr, nullptr, nb, n_tokens[i], lin, (size_t)bt, i, 0});
      lin += align_up((uint64_t)n_tokens[i] * bpt, kArenaGranule);
      bt += align_up((uint64_t)nb * 4, 16);
    }
    Plan pl;
    plan_staged(p, items, ring, resume != 0, nullptr, pl);
    int64_t n_copies = 0;
    for (auto &ch : pl.chunks) n_copies += (int64_t)ch.copies.size();
    counts[0] = (int64_t)pl.chunks.size(); counts[1] = n_copies; counts[2] = (int64_t)pl.segs.size(); counts[3] = pl.next_slot;
    if ((int64_t)pl.chunks.size() > cap || n_copies > cap || (int64_t)pl.segs.size() > cap) return fail(KVR_ERR_INVALID_ARG, "kvr_test_plan: output arrays too small");
    int64_t c = 0;
    for (size_t k = 0; k < pl.chunks.size(); ++k) {
      const Chunk &ch = pl.chunks[k];
      int64_t *o = chunks + 6 * k;
      o[0] = ch.first_slot; o[1] = ch.n_slots; o[2] = (int64_t)ch.bytes; o[3] = (int64_t)ch.copies.size(); o[4] = (int64_t)ch.seg_begin; o[5] = ch.nsegs;
      for (auto &cp : ch.copies) {
        int64_t *q = copies + 5 * c++;
        q[0] = (int64_t)k; q[1] = (int64_t)cp.lin_off; q[2] = (int64_t)cp.ring_off; q[3] = (int64_t)cp.vpos; q[4] = (int64_t)cp.bytes;
      }
    }
    for (size_t i = 0; i < pl.segs.size(); ++i) {
      const Seg &sg = pl.segs[i];
      int64_t *o = segs + 5 * i;
      o[0] = (int64_t)reinterpret_cast<uintptr_t>(sg.bt);          // the item's table offset identifies the item
      o[1] = (int64_t)(sg.img - ring.base);                        // where image byte 0 would lie, relative to the ring
      o[2] = sg.tile_begin; o[3] = sg.tile_count; o[4] = sg.nb;
    }
    return KVR_OK;
  } catch (const std::bad_alloc &) {
    return fail(KVR_ERR_NOMEM, "out of host memory");
  }
}

int32_t kvr_pool_numa_node(kvr_pool *p) { return p ? p->numa_node : -1; }

kvr_status kvr_selftest_bounded_wait(kvr_pool *p, int32_t leave_error_set) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (p->meta_only) return fail(KVR_ERR_BAD_STATE, "metadata-only pool has no device side");
  if (kvr_status s = wait_unlocked(p, enter.lock, 0, false, 60000)) return s;
  cudaError_t e = launch_wait_limit_probe(p->status_word, 4096, p->s_gather);
  if (e != cudaSuccess) return fail(KVR_ERR_CUDA, "probe launch: %s", cudaGetErrorString(e));
  CU(cudaStreamSynchronize(p->s_gather));
  const int seen = *(volatile int *)p->status_word;
  if (!leave_error_set) *p->status_word = 0;
  if (seen != 2) return fail(KVR_ERR_CUDA, "the bounded wait did not run out (status word %d)", seen);
  return KVR_OK;
}

kvr_status kvr_selftest_block_check(kvr_pool *p, int32_t leave_error_set) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (p->meta_only || !p->staging || p->NB < 2) return fail(KVR_ERR_BAD_STATE, "needs a pool with staging memory and at least two blocks");
  if (kvr_status s = wait_unlocked(p, enter.lock, 0, false, 60000)) return s;
  DescLease lease(p);
  if (kvr_status s = lease.take(enter.lock)) return s;
  if (lease.idx < 0) return fail(KVR_ERR_BAD_STATE, "no descriptor buffer free");
  DescBuf &db = p->descs[lease.idx];
  // One tile of one request whose table names the pool's last block, handed to the mover with a pool that claims
  // to be one block shorter: the entry is out of range for the kernel, yet inside the real allocation, so even a
  // broken check could not make the launch touch memory that is not the pool's.
  reinterpret_cast<int32_t *>(db.h)[0] = p->NB - 1;
  *reinterpret_cast<unsigned long long *>(db.h + 32) = 0;          // the launch's work counter
  Seg sg{};
  sg.bt = reinterpret_cast<const int32_t *>(db.d);
  sg.img = p->out_ring.base;
  sg.n_tokens = p->BS; sg.tile_begin = 0; sg.tile_count = 1; sg.nb = 1;
  memcpy(db.h + 64, &sg, sizeof sg);
  CU(cudaMemcpyAsync(db.d, db.h, 64 + sizeof sg, cudaMemcpyHostToDevice, p->s_gather));
  MoveArgs a{};
  a.segs = reinterpret_cast<const Seg *>(db.d + 64); a.nsegs = 1; a.total_tiles = 1;
  a.pool = p->d_pool; a.plane_stride = p->plane_stride; a.block_stride = p->block_stride; a.tile_bytes = p->tile_bytes;
  a.row_bytes = p->row; a.block_size = p->BS; a.num_blocks = p->NB - 1; a.status = p->status_word;
  a.work = reinterpret_cast<unsigned long long *>(db.d + 32);
  cudaError_t e = p->cfg.kernel == KVR_KERNEL_BULK ? launch_move_bulk(true, a, p->bulk, 1, p->sm_count, p->s_gather)
                                                   : launch_move_warp(true, a, 1, p->sm_count, p->s_gather);
  if (e != cudaSuccess) return fail(KVR_ERR_CUDA, "self-test launch: %s", cudaGetErrorString(e));
  CU(cudaStreamSynchronize(p->s_gather));
  const int seen = *(volatile int *)p->status_word;
  if (!leave_error_set) *p->status_word = 0;
  if (seen != kStatusBadBlock) return fail(KVR_ERR_CUDA, "the out-of-range table entry was not caught (status word %d)", seen);
  return KVR_OK;
}

kvr_status kvr_clear_device_error(kvr_pool *p) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (p->status_word) *p->status_word = 0;
  return KVR_OK;
}

kvr_status kvr_probe_link(kvr_pool *p, uint64_t bytes, int32_t reps, double *d2h_gbs, double *h2d_gbs) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (p->meta_only || !p->h_arena) return fail(KVR_ERR_BAD_STATE, "the pool has no arena to probe");
  if (reps < 1 || reps > 1000 || bytes < 4096) return fail(KVR_ERR_INVALID_ARG, "reps in [1, 1000], bytes >= 4096");
  if (kvr_status s = wait_unlocked(p, enter.lock, 0, false, 60000)) return s;
  if (p->arena.used() != 0) return fail(KVR_ERR_BAD_STATE, "the probe overwrites the arena: it must hold no image");
  if (bytes > p->arena.capacity()) bytes = p->arena.capacity() / 4096 * 4096;
  // the device end of the copies: the staging memory when it is large enough (nothing is in flight), else a
  // temporary buffer
  char *dev = nullptr;
  bool temp = false;
  if (p->staging && bytes <= p->staging_total) dev = p->staging;
  else {
    cudaError_t e = cudaMalloc((void **)&dev, bytes);
    if (e != cudaSuccess) return fail(KVR_ERR_NOMEM, "cudaMalloc(probe, %llu): %s", (unsigned long long)bytes, cudaGetErrorString(e));
    temp = true;
  }
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  kvr_status st = KVR_OK;
  auto run = [&](bool to_host, double *out) -> kvr_status {
    double best_ms = 1e30;
    for (int i = 0; i < reps + 2; ++i) {                     // two warm-ups
      cudaStream_t s = to_host ? p->s_d2h : p->s_h2d;
      CU(cudaEventRecord(e0, s));
      if (to_host) CU(cudaMemcpyAsync(p->h_arena, dev, bytes, cudaMemcpyDefault, s));
      else CU(cudaMemcpyAsync(dev, p->h_arena, bytes, cudaMemcpyDefault, s));
      CU(cudaEventRecord(e1, s));
      CU(cudaEventSynchronize(e1));
      float ms = 0;
      CU(cudaEventElapsedTime(&ms, e0, e1));
      if (i >= 2 && ms < best_ms) best_ms = ms;
    }
    if (out) *out = (double)bytes / best_ms / 1e6;
    return KVR_OK;
  };
  if ((st = get_event(p, &e0)) == KVR_OK && (st = get_event(p, &e1)) == KVR_OK &&
      (st = run(true, d2h_gbs)) == KVR_OK)
    st = run(false, h2d_gbs);
  put_event(p, e0); put_event(p, e1);
  if (temp) cudaFree(dev);
  return st;
}

kvr_status kvr_read_load(const void *device_buf, uint64_t bytes, int32_t launches, void *device_sink, void *stream) {
  if (!device_buf || !device_sink || bytes < 16 || launches < 0 || ((uintptr_t)device_buf & 15) || ((uintptr_t)device_sink & 7))
    return fail(KVR_ERR_INVALID_ARG, "kvr_read_load: NULL, misaligned or empty buffer");
  cudaError_t e = launch_read_load(device_buf, bytes, launches, device_sink, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail(KVR_ERR_CUDA, "read load launch: %s", cudaGetErrorString(e));
  return KVR_OK;
}

void *kvr_pool_device_ptr(kvr_pool *p) { return p ? p->d_pool : nullptr; }
void *kvr_pool_host_arena(kvr_pool *p) { return p ? p->h_arena : nullptr; }

}  // extern "C"
