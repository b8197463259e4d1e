// Transfer engine of the KV retention mover: streams, staging rings, the chunk planner and the move queue.
//
// Every batch call settles the bookkeeping at once (states, block tables, arena
// offsets: the same answers a synchronous implementation gives) and enqueues
// the byte movement on four streams:
//
//   suspend, staged route :  gather kernel -> staging ring    (s_gather)
//                            ring -> pinned arena, DMA        (s_d2h)
//   resume,  staged route :  pinned arena -> ring, DMA        (s_h2d)
//                            scatter kernel ring -> pool      (s_scatter)
//   mapped route          :  the kernel reads / writes the arena itself
//
// so a suspend and a resume use different streams and different staging rings
// and can overlap, one per link direction.  Hazards between calls are ordered
// on the device with events, not by blocking the caller:
//   - a block read by a suspend's gather carries that move's sequence number; whoever
//     takes the block next waits for that move's gather ("read_done");
//   - a host range freed by a resume is remembered with the move's sequence
//     number; a suspend that lands on it waits for the move's last read;
//   - a move on a request whose previous move is in flight waits for it.
//
// A staging ring is `slots` slots of `slot_bytes`.  One mover launch ("chunk") covers up to slots - 1 consecutive
// slots, wrapping around the ring's end; each slot is handed back by its own event as soon as its bytes have left
// (suspend) or have been scattered (resume), so the next launch can start while the link still drains the last slot
// of the previous one.  Launches are therefore almost as large as the ring, which matters because every launch
// pays a fixed completion latency while the copy engine is busy.
#include "kvr_pool.hpp"

namespace kvr {

namespace {
thread_local std::string g_err;
}

kvr_status fail(kvr_status st, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return st;
}

// lets the library's other source files report through kvr_last_error()
void set_last_error(const char *msg) { g_err = msg ? msg : ""; }
const char *last_error_text() { return g_err.c_str(); }

// ---- events, descriptors, op tracking ----------------------------------------------------

kvr_status get_event(kvr_pool *p, cudaEvent_t *out) {
  if (!p->event_pool.empty()) { *out = p->event_pool.back(); p->event_pool.pop_back(); return KVR_OK; }
  CUP(p, cudaEventCreate(out));
  return KVR_OK;
}
void put_event(kvr_pool *p, cudaEvent_t e) { if (e) p->event_pool.push_back(e); }

static kvr_status new_desc(size_t cap, DescBuf *b) {
  b->cap = cap;
  CU(cudaHostAlloc((void **)&b->h, b->cap, cudaHostAllocDefault));
  cudaError_t e = cudaMalloc((void **)&b->d, b->cap);
  if (e != cudaSuccess) { cudaFreeHost(b->h); b->h = nullptr; return fail(KVR_ERR_NOMEM, "cudaMalloc(descriptors): %s", cudaGetErrorString(e)); }
  return KVR_OK;
}

static void free_desc(DescBuf &b) {
  if (b.h) cudaFreeHost(b.h);
  if (b.d) cudaFree(b.d);
  b = DescBuf();
}

static void retire(kvr_pool *p, Op &op) {
  for (auto &rd : op.reqs) {
    auto it = p->reqs.find(rd.id);
    if (it == p->reqs.end() || it->second.pending_op != op.seq) continue;
    Request &r = it->second;
    r.pending_op = 0; r.pending_kind = 0;
    float ms = 0;
    cudaEvent_t last = rd.chunk >= 0 ? op.chunk_done[rd.chunk] : op.start;
    if (cudaEventElapsedTime(&ms, op.start, last) == cudaSuccess) {
      r.has_latency = true; r.host_ms = op.host_ms; r.device_ms = ms;
    }
  }
  for (auto &pr : op.prof) {
    float ms = 0;
    if (cudaEventElapsedTime(&ms, pr.first, pr.second) == cudaSuccess) {
      if (op.kind == OP_SUSPEND || op.kind == OP_EXPORT) p->st.gather_ms += ms; else p->st.scatter_ms += ms;
    }
    put_event(p, pr.first); put_event(p, pr.second);
  }
  if (op.desc >= 0 && op.n_stamps) {
    // first CTA start to last CTA end of every launch, as the kernels stamped them
    const LaunchRec *rec = reinterpret_cast<const LaunchRec *>(p->descs[op.desc].h + op.stamp_off);
    double ms = 0;
    for (int i = 0; i < op.n_stamps; ++i)
      if (rec[i].last_end > rec[i].first_start) ms += (double)(rec[i].last_end - rec[i].first_start) * 1e-6;
    if (op.kind == OP_SUSPEND || op.kind == OP_EXPORT) p->st.gather_kernel_ms += ms; else p->st.scatter_kernel_ms += ms;
  }
  for (auto e : op.chunk_done) put_event(p, e);
  for (auto e : op.aux) put_event(p, e);
  put_event(p, op.start); put_event(p, op.read_done); put_event(p, op.done);
  if (op.desc >= 0) {
    if (p->descs[op.desc].one_off) free_desc(p->descs[op.desc]); else p->descs[op.desc].busy = 0;
  }
}

// retire every move whose last event has fired
kvr_status poll(kvr_pool *p) {
  for (auto it = p->ops.begin(); it != p->ops.end();) {
    cudaError_t e = cudaEventQuery(it->second.done);
    if (e == cudaSuccess) { retire(p, it->second); it = p->ops.erase(it); }
    else if (e == cudaErrorNotReady) ++it;
    else return fail(KVR_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
  }
  if (!p->pending_free.empty()) {
    size_t k = 0;
    for (auto &pf : p->pending_free) if (p->ops.count(pf.seq)) p->pending_free[k++] = pf;
    p->pending_free.resize(k);
  }
  return KVR_OK;
}

// one look at a move (seq) or at all moves (seq = 0): KVR_OK when it has landed (read_only: when its source is no
// longer read), KVR_ERR_TIMEOUT when it is still in flight
kvr_status look(kvr_pool *p, uint64_t seq, bool read_only) {
  if (read_only && seq) {
    auto it = p->ops.find(seq);
    if (it == p->ops.end()) return KVR_OK;
    cudaError_t e = cudaEventQuery(it->second.read_done);
    if (e == cudaSuccess) return KVR_OK;
    if (e != cudaErrorNotReady) return fail(KVR_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
    return KVR_ERR_TIMEOUT;
  }
  if (kvr_status s = poll(p)) return s;
  if (seq ? p->ops.count(seq) : !p->ops.empty()) return KVR_ERR_TIMEOUT;
  if (p->status_word && *(volatile int *)p->status_word != 0)
    return fail(KVR_ERR_CUDA, "a mover gave up on a bounded wait (status %d)", *(volatile int *)p->status_word);
  return KVR_OK;
}

// Bounded host-side wait for one move (seq) or all (seq = 0).  The pool's lock (held on entry and on return) is
// given up while the thread sleeps, so other callers keep working on the pool; whatever the caller knew about
// requests before the wait must be looked up again afterwards.
kvr_status wait_unlocked(kvr_pool *p, std::unique_lock<std::mutex> &lock, uint64_t seq, bool read_only, int64_t timeout_ms) {
  if (p->meta_only) return KVR_OK;
  if (timeout_ms < 0) timeout_ms = 60000;
  const auto t0 = Clock::now();
  for (unsigned spin = 0;; ++spin) {
    const kvr_status s = look(p, seq, read_only);
    if (s != KVR_ERR_TIMEOUT) return s;
    if (ms_since(t0) > (double)timeout_ms) return fail(KVR_ERR_TIMEOUT, "move still in flight after %lld ms", (long long)timeout_ms);
    lock.unlock();
    if (spin > 2000) std::this_thread::sleep_for(std::chrono::microseconds(50)); else std::this_thread::yield();
    lock.lock();
  }
}

// the same wait with the lock held throughout (pool destruction, self-tests)
kvr_status wait_locked(kvr_pool *p, uint64_t seq, int64_t timeout_ms) {
  if (p->meta_only) return KVR_OK;
  const auto t0 = Clock::now();
  for (unsigned spin = 0;; ++spin) {
    const kvr_status s = look(p, seq, false);
    if (s != KVR_ERR_TIMEOUT) return s;
    if (ms_since(t0) > (double)timeout_ms) return fail(KVR_ERR_TIMEOUT, "move still in flight after %lld ms", (long long)timeout_ms);
    if (spin > 2000) std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
}

// make stream s wait for a move's event, if the move is still in flight
kvr_status stream_after(kvr_pool *p, cudaStream_t s, uint64_t seq, bool read_only) {
  if (!seq) return KVR_OK;
  auto it = p->ops.find(seq);
  if (it == p->ops.end()) return KVR_OK;
  CUP(p, cudaStreamWaitEvent(s, read_only ? it->second.read_done : it->second.done, 0));
  return KVR_OK;
}


// Size limit of the next chunk of a staged move, given how many bytes earlier chunks hold and how many the move has
// in all.  Every launch costs tens of microseconds of latency besides its bytes, so a move wants few, large
// launches; what speaks against one single launch is latency at the link: a suspend's first byte crosses only after
// the first gather, and a resume's last scatter starts only after the last byte has arrived.  The movers are ~50
// times faster than the link, so it is enough to keep the first chunk of a suspend and the last chunk of a resume
// small -- one staging slot -- and let every other chunk be as large as the ring allows (`big`):
//   suspend: [slot] [big] [big] ... [rest];      resume: [big] [big] ... [rest - slot] [slot].
// Below a size threshold the split is not worth a launch and the move goes in one: 1 GiB for a suspend (its blocks
// are free 0.35 ms later, 2 % of the move), 256 MiB for a resume (at most 85 us between the last byte and a usable
// request: a resume's latency is what the caller waits for).
static uint64_t next_cap(const kvr_pool *p, uint64_t done, uint64_t total, bool resume, uint64_t big) {
  const uint64_t tile = (uint64_t)p->tile_bytes, slot = p->slot_bytes;
  const uint64_t left = total > done ? total - done : 0;
  uint64_t cap = big;
  if (total > (resume ? p->resume_single : p->suspend_single) && total > 2 * slot) {
    if (!resume) { if (done == 0) cap = slot; }
    else if (left > 2 * slot && left <= big + slot) cap = left - slot;
  }
  if (cap > big) cap = big;
  if (cap < tile) cap = tile;
  return cap;
}

// Staged route: cut the concatenated images into chunks on tile boundaries.  A chunk starts on a slot boundary of
// the ring and runs over consecutive slots; positions inside it are "virtual" bytes counted from its start, the
// physical offset being (first_slot * slot + v) mod ring size.  Where the ring wraps, the run of tiles in progress
// ends and a new segment starts at offset 0 (the few bytes before the end that hold no whole tile stay unused and
// count as virtual bytes), so every segment is linear in memory and the kernels never see the wrap.
void plan_staged(kvr_pool *p, const std::vector<Item> &items, Ring &ring, bool ramp_down_too, const char *desc_dev, Plan &pl) {
  uint64_t total = 0;
  for (auto &it : items) total += (uint64_t)it.n_tokens * p->bpt;
  const uint64_t slot = p->slot_bytes, n = ring.slots.size(), S = slot * n, big = slot * (uint64_t)p->launch_slots;
  int first = ring.next;
  Chunk cur;
  uint64_t vfill = 0, payload = 0, done = 0, cap = 0;
  auto open = [&]() {
    cur = Chunk();
    cur.first_slot = first;
    cur.seg_begin = pl.segs.size();
    vfill = payload = 0;
    cap = next_cap(p, done, total, ramp_down_too, big);
  };
  auto flush = [&]() {
    if (cur.nsegs) {
      cur.bytes = payload;
      cur.n_slots = (int)((vfill + slot - 1) / slot);
      done += payload;
      first = (first + cur.n_slots) % (int)n;
      alloc_point(p);
      pl.chunks.push_back(cur);
    }
    open();
  };
  open();
  pl.req_chunk.assign(items.size(), -1);
  for (size_t i = 0; i < items.size(); ++i) {
    const Item &it = items[i];
    const long long T = (long long)p->planes * it.nb;
    const uint64_t img_bytes = (uint64_t)it.n_tokens * p->bpt;
    long long q0 = 0;
    while (q0 < T) {
      const uint64_t at = ((uint64_t)cur.first_slot * slot + vfill) % S;   // physical offset of the next byte
      const uint64_t to_end = S - at, left = cap - vfill;
      const uint64_t room = left < to_end ? left : to_end;
      const uint64_t base = tile_off(p, it, q0);
      long long lo = q0, hi = T;           // largest q1 with tile_off(q1) - base <= room
      while (lo < hi) {
        const long long mid = (lo + hi + 1) >> 1;
        const uint64_t end = mid == T ? img_bytes : tile_off(p, it, mid);
        if (end - base <= room) lo = mid; else hi = mid - 1;
      }
      if (lo == q0 || cur.nsegs == kMaxSegs) {
        const uint64_t one = (q0 + 1 == T ? img_bytes : tile_off(p, it, q0 + 1)) - base;
        if (lo == q0 && cur.nsegs != kMaxSegs && to_end < left && left - to_end >= one) { vfill += to_end; continue; }   // skip to the ring's start
        flush();
        continue;
      }
      const long long q1 = lo;
      const uint64_t end = q1 == T ? img_bytes : tile_off(p, it, q1);
      const uint64_t bytes = end - base;
      Seg sg{};
      sg.bt = reinterpret_cast<const int32_t *>(desc_dev + it.bt_off);
      sg.img = ring.base + at - base;
      sg.n_tokens = it.n_tokens; sg.tile_begin = q0; sg.tile_count = q1 - q0; sg.nb = it.nb;
      alloc_point(p);
      pl.segs.push_back(sg);
      cur.nsegs++; cur.tiles += q1 - q0;
      const uint64_t lin = it.lin_off + base;
      if (!cur.copies.empty() && cur.copies.back().lin_off + cur.copies.back().bytes == lin &&
          cur.copies.back().ring_off + cur.copies.back().bytes == at)
        cur.copies.back().bytes += bytes;
      else
        cur.copies.push_back({lin, at, vfill, bytes});
      vfill += bytes; payload += bytes;
      pl.req_chunk[i] = (int)pl.chunks.size();
      q0 = q1;
      if (cap - vfill < (uint64_t)p->row) flush();
    }
    // low-latency resume: close the chunk where a request ends, so the request is complete (its scatter launched)
    // as soon as its own bytes have arrived instead of waiting for the rest of a launch
    if (ramp_down_too && (p->call_flags & KVR_LOW_LATENCY) && T > 0 && cur.nsegs) flush();
  }
  flush();
  pl.next_slot = first;
}

// Direct routes (mapped arena, export / import): one linear buffer, launches of up to kMaxSegs requests.
static void plan_direct(kvr_pool *p, const std::vector<Item> &items, char *lin_base, const char *desc_dev, Plan &pl) {
  Chunk cur;
  cur.seg_begin = 0;
  pl.req_chunk.assign(items.size(), -1);
  for (size_t i = 0; i < items.size(); ++i) {
    const Item &it = items[i];
    const long long T = (long long)p->planes * it.nb;
    if (T == 0) continue;
    if (cur.nsegs == kMaxSegs) { pl.chunks.push_back(cur); cur = Chunk(); cur.seg_begin = pl.segs.size(); }
    Seg sg{};
    sg.bt = reinterpret_cast<const int32_t *>(desc_dev + it.bt_off);
    sg.img = lin_base + it.lin_off;
    sg.n_tokens = it.n_tokens; sg.tile_begin = 0; sg.tile_count = T; sg.nb = it.nb;
    alloc_point(p);
    pl.segs.push_back(sg);
    cur.nsegs++; cur.tiles += T; cur.bytes += (uint64_t)it.n_tokens * p->bpt;
    pl.req_chunk[i] = (int)pl.chunks.size();
  }
  if (cur.nsegs) pl.chunks.push_back(cur);
}

static kvr_status launch(kvr_pool *p, bool gather, const Seg *segs_dev, const Chunk &c, cudaStream_t s, Op &op,
                  LaunchRec *rec_dev) {
  MoveArgs a{};
  a.segs = segs_dev + c.seg_begin; a.nsegs = c.nsegs; a.total_tiles = c.tiles;
  a.pool = p->d_pool; a.plane_stride = p->plane_stride; a.block_stride = p->block_stride; a.tile_bytes = p->tile_bytes;
  a.row_bytes = p->row; a.block_size = p->BS; a.num_blocks = p->NB; a.status = p->status_word;
  a.stamp = p->profile ? &rec_dev->first_start : nullptr;
  a.work = &rec_dev->work;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (p->profile) {
    kvr_status s0 = get_event(p, &e0); if (s0) return s0;
    s0 = get_event(p, &e1); if (s0) { put_event(p, e0); return s0; }
    alloc_point(p);
    op.prof.push_back({e0, e1});
    CUP(p, cudaEventRecord(e0, s));
  }
  if (inject_cuda(p)) return fail(KVR_ERR_CUDA, "injected failure of the mover launch");
  cudaError_t e = p->cfg.kernel == KVR_KERNEL_BULK
                      ? launch_move_bulk(gather, a, p->bulk, p->cfg.max_ctas, p->sm_count, s)
                      : launch_move_warp(gather, a, p->cfg.max_ctas, p->sm_count, s);
  if (e != cudaSuccess) return fail(KVR_ERR_CUDA, "mover launch: %s", cudaGetErrorString(e));
  if (p->profile) CUP(p, cudaEventRecord(e1, s));
  if (gather) { p->st.gather_launches++; p->st.gather_bytes += c.bytes; }
  else { p->st.scatter_launches++; p->st.scatter_bytes += c.bytes; }
  return KVR_OK;
}

// the move is completely enqueued: make it visible on its requests (nothing here can fail)
static void register_op(Op &op, std::vector<Item> &items, const std::vector<int> &req_chunk, int kind,
                 Clock::time_point t_call, uint64_t *out_seq) {
  op.host_ms = ms_since(t_call);
  for (size_t i = 0; i < items.size(); ++i) {
    op.reqs[i] = {items[i].id, req_chunk[i]};
    if (items[i].r) {
      items[i].r->pending_op = op.seq;
      items[i].r->pending_kind = kind == OP_SUSPEND ? KVR_SUSPENDING : kind == OP_RESUME ? KVR_RESUMING : 0;
      items[i].r->has_latency = false;
    }
  }
  *out_seq = op.seq;
}

// Strided-copy route: no kernel and no staging.  For every block, one cudaMemcpy2DAsync moves its 2L tiles
// (rows of `width` valid bytes, `plane_stride` apart in the pool, one image plane apart in the arena).
static kvr_status enqueue_dma2d(kvr_pool *p, Op &op, std::vector<Item> &items, bool to_linear, uint64_t block_tag,
                         const std::vector<uint64_t> &arena_waits, Clock::time_point t_call, uint64_t *out_seq) {
  cudaStream_t c = to_linear ? p->s_d2h : p->s_h2d;
  kvr_status s;
  CUP(p, cudaEventRecord(op.start, c));
  for (auto &it : items)
    if (it.r && it.r->pending_op && (s = stream_after(p, c, it.r->pending_op, false))) return s;
  if (!to_linear && (s = stream_after(p, c, block_tag, true))) return s;
  for (uint64_t w : arena_waits) if ((s = stream_after(p, c, w, true))) return s;
  std::vector<int> req_chunk(items.size(), -1);
  for (size_t i = 0; i < items.size(); ++i) {
    const Item &it = items[i];
    if (!it.nb) continue;
    const size_t img_pitch = (size_t)it.n_tokens * p->row;
    for (int32_t b = 0; b < it.nb; ++b) {
      long long valid = it.n_tokens - (long long)b * p->BS;
      if (valid > p->BS) valid = p->BS;
      const size_t width = (size_t)valid * p->row;
      char *pool_ptr = p->d_pool + (long long)it.blocks[b] * p->block_stride;
      char *img_ptr = p->h_arena + it.lin_off + (size_t)b * p->BS * p->row;
      if (to_linear) {
        CUP(p, cudaMemcpy2DAsync(img_ptr, img_pitch, pool_ptr, (size_t)p->plane_stride, width, (size_t)p->planes, cudaMemcpyDefault, c));
        p->st.d2h_copies++; p->st.d2h_bytes += width * p->planes;
      } else {
        CUP(p, cudaMemcpy2DAsync(pool_ptr, (size_t)p->plane_stride, img_ptr, img_pitch, width, (size_t)p->planes, cudaMemcpyDefault, c));
        p->st.h2d_copies++; p->st.h2d_bytes += width * p->planes;
      }
    }
    cudaEvent_t cd;
    if ((s = get_event(p, &cd))) return s;
    alloc_point(p);
    op.chunk_done.push_back(cd);
    CUP(p, cudaEventRecord(cd, c));
    req_chunk[i] = (int)op.chunk_done.size() - 1;
  }
  CUP(p, cudaEventRecord(op.read_done, c));
  CUP(p, cudaEventRecord(op.done, c));
  register_op(op, items, req_chunk, op.kind, t_call, out_seq);
  return KVR_OK;
}

// Build and upload the descriptors of a move, then enqueue it.  `to_linear` = gather direction.
// route: KVR_ROUTE_STAGED, KVR_ROUTE_MAPPED, KVR_ROUTE_DMA2D, or 0 for a caller-supplied device buffer (lin_dev).
static kvr_status enqueue_impl(kvr_pool *p, Op &op, int kind, std::vector<Item> &items, int route, char *lin_dev,
                        uint64_t block_tag, const std::vector<uint64_t> &arena_waits, Clock::time_point t_call,
                        int lease, uint64_t *out_seq) {
  const bool to_linear = (kind == OP_SUSPEND || kind == OP_EXPORT);
  kvr_status s = KVR_OK;
  if ((s = get_event(p, &op.start)) || (s = get_event(p, &op.read_done)) || (s = get_event(p, &op.done))) return s;
  alloc_point(p);
  op.reqs.resize(items.size());

  if (route == KVR_ROUTE_DMA2D) return enqueue_dma2d(p, op, items, to_linear, block_tag, arena_waits, t_call, out_seq);

  // plan with table addresses relative to the descriptor buffer, then size the buffer exactly:
  // [block tables][segments][one record per launch: work counter and time stamps]
  size_t bt_bytes = 0;
  for (auto &it : items) { it.bt_off = bt_bytes; bt_bytes += align_up((uint64_t)it.nb * 4, 16); }
  Plan pl;
  Ring *ring = nullptr;
  if (route == KVR_ROUTE_STAGED) {
    ring = to_linear ? &p->out_ring : &p->in_ring;
    plan_staged(p, items, *ring, !to_linear, nullptr, pl);
  } else {
    plan_direct(p, items, route == KVR_ROUTE_MAPPED ? p->arena_dev : lin_dev, nullptr, pl);
  }
  const size_t seg_off = align_up(bt_bytes, 64);
  const size_t rec_off = align_up(seg_off + pl.segs.size() * sizeof(Seg), 64);
  const int n_recs = (int)pl.chunks.size();
  size_t desc_bytes = rec_off + sizeof(LaunchRec) * (size_t)n_recs;
  if (!desc_bytes) desc_bytes = 64;
  if (lease >= 0 && p->descs[lease].cap >= desc_bytes) {
    op.desc = lease;
  } else {
    // more descriptors than a pre-sized buffer holds: a one-off buffer, freed when the move retires
    alloc_point(p);
    size_t slot_i = p->descs.size();
    for (size_t i = 0; i < p->descs.size(); ++i) if (!p->descs[i].h) { slot_i = i; break; }
    if (slot_i == p->descs.size()) p->descs.push_back(DescBuf());
    size_t cap = 1 << 20;
    while (cap < desc_bytes) cap <<= 1;
    if ((s = new_desc(cap, &p->descs[slot_i]))) return s;
    p->descs[slot_i].one_off = true;
    op.desc = (int)slot_i;
  }
  DescBuf &db = p->descs[op.desc];
  db.busy = op.seq;
  for (int i = 0; i < n_recs; ++i) reinterpret_cast<LaunchRec *>(db.h + rec_off)[i] = LaunchRec{~0ull, 0, 0, 0};
  op.stamp_off = rec_off; op.n_stamps = p->profile ? n_recs : 0;
  LaunchRec *recs_dev = reinterpret_cast<LaunchRec *>(db.d + rec_off);
  for (auto &it : items) if (it.nb) memcpy(db.h + it.bt_off, it.blocks, (size_t)it.nb * 4);
  for (auto &sg : pl.segs) sg.bt = reinterpret_cast<const int32_t *>(db.d + reinterpret_cast<uintptr_t>(sg.bt));
  if (!pl.segs.empty()) memcpy(db.h + seg_off, pl.segs.data(), pl.segs.size() * sizeof(Seg));
  const Seg *segs_dev = reinterpret_cast<const Seg *>(db.d + seg_off);

  // streams: `k` runs the kernel, `c` runs the copies (staged route only)
  cudaStream_t k = to_linear ? p->s_gather : p->s_scatter;
  cudaStream_t c = to_linear ? p->s_d2h : p->s_h2d;
  const bool staged = route == KVR_ROUTE_STAGED;
  cudaStream_t first = (staged && !to_linear) ? c : k;    // stream of the first byte moved
  cudaStream_t host_side = staged ? c : k;                // stream that touches the arena

  CUP(p, cudaEventRecord(op.start, first));
  // a move on a request waits for that request's previous move
  for (auto &it : items)
    if (it.r && it.r->pending_op) {
      if ((s = stream_after(p, first, it.r->pending_op, false))) return s;
      if (first != k && (s = stream_after(p, k, it.r->pending_op, false))) return s;
    }
  // blocks handed to a scatter may still be read by an earlier gather
  if (!to_linear && (s = stream_after(p, k, block_tag, true))) return s;
  // host ranges handed to a suspend may still be read by an earlier resume
  for (uint64_t w : arena_waits) if ((s = stream_after(p, host_side, w, true))) return s;

  CUP(p, cudaMemcpyAsync(db.d, db.h, desc_bytes, cudaMemcpyHostToDevice, k));
  p->st.desc_bytes += desc_bytes;

  // size of one link copy: copy_piece (64 MiB), or more when the move is so large (beyond 64 GiB) that such pieces
  // would put thousands of entries into the copy stream (a full stream queue blocks the caller, and with it the
  // next call's overlap).  A copy never crosses a cut point: with pieces no larger than a slot the cut points are
  // the slot boundaries and every `piece` bytes inside a slot -- so a resume's first copy of a launch fits the
  // ring's one free slot and runs while the previous launch is still being scattered -- otherwise every whole
  // number of slots that fits a piece.
  const uint64_t slot = p->slot_bytes;
  uint64_t piece = p->copy_piece;
  {
    uint64_t total = 0;
    for (auto &ch : pl.chunks) total += ch.bytes;
    const uint64_t floor_piece = align_up(total / 512 + 1, 1 << 20);
    if (piece < floor_piece) piece = floor_piece;
  }
  // next cut point after virtual position v of a chunk of n_slots slots
  auto next_cut = [&](uint64_t v, int n_slots) -> uint64_t {
    if (piece < 2 * slot) {                       // pieces within a slot
      const uint64_t step = piece < slot ? piece : slot;
      const uint64_t slot_end = (v / slot + 1) * slot, o = v % slot;
      const uint64_t nx = v - o + (o / step + 1) * step;
      return nx < slot_end ? nx : slot_end;
    }
    const uint64_t G = piece / slot * slot;       // pieces of whole slots
    if (to_linear) {                              // ... with a cut where all slots but the last are done (early release)
      const uint64_t early = (uint64_t)(n_slots - 1) * slot;
      const uint64_t nx = (v / G + 1) * G;
      return (v < early && nx > early) ? early : nx;
    }
    if (v < slot) return slot;                    // ... after a first copy that fits the ring's one free slot
    return slot + ((v - slot) / G + 1) * G;
  };
  const int n_ring = ring ? (int)ring->slots.size() : 1;
  for (size_t ci = 0; ci < pl.chunks.size(); ++ci) {
    const Chunk &ch = pl.chunks[ci];
    cudaEvent_t cd;
    if ((s = get_event(p, &cd))) return s;
    alloc_point(p);
    op.chunk_done.push_back(cd);
    if (!staged) {
      if ((s = launch(p, to_linear, segs_dev, ch, k, op, recs_dev + ci))) return s;
      CUP(p, cudaEventRecord(cd, k));
      continue;
    }
    cudaEvent_t filled;
    if ((s = get_event(p, &filled))) return s;
    alloc_point(p);
    op.aux.push_back(filled);
    // hand a run of the chunk's slots [j0, j1) back with one event, recorded on stream `on` in the last slot of the run
    auto release = [&](int j0, int j1, cudaStream_t on) -> kvr_status {
      const int owner = (ch.first_slot + j1 - 1) % n_ring;
      CUP(p, cudaEventRecord(ring->slots[owner].freed, on));
      const uint64_t q = ++ring->seq;
      for (int j = j0; j < j1; ++j) {
        Slot &sl = ring->slots[(ch.first_slot + j) % n_ring];
        sl.used = true; sl.seq = q; sl.owner = owner;
      }
      return KVR_OK;
    };
    if (to_linear) {
      // the launch writes all of its slots at once: wait for the latest release among them (it covers the others)
      const Slot *latest = nullptr;
      for (int j = 0; j < ch.n_slots; ++j) {
        const Slot &sl = ring->slots[(ch.first_slot + j) % n_ring];
        if (sl.used && (!latest || sl.seq > latest->seq)) latest = &sl;
      }
      if (latest) CUP(p, cudaStreamWaitEvent(k, ring->slots[latest->owner].freed, 0));
      if ((s = launch(p, true, segs_dev, ch, k, op, recs_dev + ci))) return s;
      CUP(p, cudaEventRecord(filled, k));
      CUP(p, cudaStreamWaitEvent(c, filled, 0));
      // the copies go out in pieces: one very large cudaMemcpyAsync to pinned memory sustains less than the same
      // bytes in 64 MiB calls on some hosts (51.5 vs 56.3 GB/s measured), and never more.  All slots but the last
      // are handed back as soon as the copies that read them are queued -- that is what the next launch, which
      // takes the ring's one free slot and those, is waiting for -- and the last one at the end.
      const int early = ch.n_slots - 1;
      bool early_done = early == 0;
      for (auto &cp : ch.copies)
        for (uint64_t o = 0; o < cp.bytes;) {
          const uint64_t v = cp.vpos + o;
          uint64_t nbytes = next_cut(v, ch.n_slots) - v;
          if (nbytes > cp.bytes - o) nbytes = cp.bytes - o;
          CUP(p, cudaMemcpyAsync(p->h_arena + cp.lin_off + o, ring->base + cp.ring_off + o, nbytes, cudaMemcpyDefault, c));
          p->st.d2h_copies++; p->st.d2h_bytes += nbytes;
          o += nbytes;
          if (!early_done && (uint64_t)early * slot <= cp.vpos + o) {
            if ((s = release(0, early, c))) return s;
            early_done = true;
          }
        }
      if ((s = release(early_done ? early : 0, ch.n_slots, c))) return s;
      CUP(p, cudaEventRecord(cd, c));
    } else {
      // the copies fill the slots one after another: each waits only for the release of the slots it touches, so
      // the link keeps running into the ring's free slot while the previous launch still scatters out of the others
      uint64_t waited_seq = 0;
      int looked = 0;
      for (auto &cp : ch.copies)
        for (uint64_t o = 0; o < cp.bytes;) {
          const uint64_t v = cp.vpos + o;
          uint64_t nbytes = next_cut(v, ch.n_slots) - v;
          if (nbytes > cp.bytes - o) nbytes = cp.bytes - o;
          for (; looked < ch.n_slots && (uint64_t)looked * slot < v + nbytes; ++looked) {
            const Slot &sl = ring->slots[(ch.first_slot + looked) % n_ring];
            if (sl.used && sl.seq > waited_seq) {
              CUP(p, cudaStreamWaitEvent(c, ring->slots[sl.owner].freed, 0));
              waited_seq = sl.seq;
            }
          }
          CUP(p, cudaMemcpyAsync(ring->base + cp.ring_off + o, p->h_arena + cp.lin_off + o, nbytes, cudaMemcpyDefault, c));
          p->st.h2d_copies++; p->st.h2d_bytes += nbytes;
          o += nbytes;
        }
      CUP(p, cudaEventRecord(filled, c));
      CUP(p, cudaStreamWaitEvent(k, filled, 0));
      if ((s = launch(p, false, segs_dev, ch, k, op, recs_dev + ci))) return s;
      if ((s = release(0, ch.n_slots, k))) return s;       // the scatter has read every slot of the chunk
      CUP(p, cudaEventRecord(cd, k));
    }
  }

  // read_done: the source of the move is no longer read.  done: the last byte has landed.
  cudaStream_t last = staged ? (to_linear ? c : k) : k;
  cudaStream_t reader = staged ? (to_linear ? k : c) : k;
  CUP(p, cudaEventRecord(op.read_done, reader));
  if (first != last) CUP(p, cudaStreamWaitEvent(last, op.read_done, 0));   // `done` must also cover the first stream (e.g. an empty move)
  if (op.n_stamps)   // the stamps come back with the move: `last` is ordered after every launch
    CUP(p, cudaMemcpyAsync(db.h + rec_off, db.d + rec_off, sizeof(LaunchRec) * (size_t)n_recs, cudaMemcpyDeviceToHost, last));
  CUP(p, cudaEventRecord(op.done, last));

  if (staged) ring->next = pl.next_slot;
  register_op(op, items, pl.req_chunk, kind, t_call, out_seq);
  return KVR_OK;
}

// A move could not be enqueued completely.  Part of it may already sit in the streams: wait for that work (it
// touches only staging memory, the arena range and the blocks the caller is about to take back), so that nothing of
// it is in flight when the bookkeeping is rolled back, then start the rings afresh.
static void drain(kvr_pool *p) {
  for (cudaStream_t s : {p->s_gather, p->s_d2h, p->s_h2d, p->s_scatter}) if (s) cudaStreamSynchronize(s);
  cudaGetLastError();
  for (Ring *r : {&p->out_ring, &p->in_ring}) {
    for (auto &sl : r->slots) sl.used = false;
    r->next = 0;
  }
}

// after drain(): every event of the abandoned move has fired or was never recorded, so all of them can be reused
static void abandon(kvr_pool *p, Op &op) {
  for (auto &pr : op.prof) { put_event(p, pr.first); put_event(p, pr.second); }
  for (auto e : op.chunk_done) put_event(p, e);
  for (auto e : op.aux) put_event(p, e);
  for (cudaEvent_t e : {op.start, op.read_done, op.done}) put_event(p, e);
  if (op.desc >= 0) {
    if (p->descs[op.desc].one_off) free_desc(p->descs[op.desc]); else p->descs[op.desc].busy = kLeased;   // back to the caller's lease
  }
}

kvr_status enqueue(kvr_pool *p, int kind, std::vector<Item> &items, int route, char *lin_dev, uint64_t block_tag,
                   const std::vector<uint64_t> &arena_waits, Clock::time_point t_call, int lease, uint64_t *out_seq) {
  if (kvr_status s = poll(p)) return s;
  const uint64_t seq = p->next_seq;
  alloc_point(p);
  Op &op = p->ops[seq];                 // the map node exists before anything is queued: registering cannot fail later
  p->next_seq++;
  op.seq = seq;
  op.kind = kind;
  kvr_status s;
  try {
    s = enqueue_impl(p, op, kind, items, route, lin_dev, block_tag, arena_waits, t_call, lease, out_seq);
  } catch (const std::bad_alloc &) {
    s = fail(KVR_ERR_NOMEM, "out of host memory while enqueueing a move");
  }
  if (s != KVR_OK) {
    drain(p);
    try { abandon(p, op); } catch (const std::bad_alloc &) {}
    p->ops.erase(seq);
  }
  return s;
}

void destroy_engine(kvr_pool *p) {
  for (auto &d : p->descs) free_desc(d);
  for (Ring *r : {&p->out_ring, &p->in_ring})
    for (auto &s : r->slots) if (s.freed) cudaEventDestroy(s.freed);
  for (auto e : p->event_pool) cudaEventDestroy(e);
  if (p->own_staging && p->staging) cudaFree(p->staging);
  if (p->status_word) cudaFreeHost(p->status_word);
  cudaStream_t *ss[4] = {&p->s_gather, &p->s_d2h, &p->s_h2d, &p->s_scatter};
  for (int i = 0; i < 4; ++i) if (p->own_stream[i] && *ss[i]) cudaStreamDestroy(*ss[i]);
  if (p->own_pool && p->d_pool) cudaFree(p->d_pool);
  if (p->own_arena && p->h_arena) {
    if (p->arena_map) { cudaHostUnregister(p->h_arena); munmap(p->arena_map, p->arena_map_len); }
    else cudaFreeHost(p->h_arena);
  }
}

// Page-locked arena of the library's own: an anonymous mapping backed by transparent huge pages where the host
// offers them, faulted in by several threads and then registered with CUDA.  Locking 2 MiB pages is several times
// quicker than cudaHostAlloc's 4 KiB pages (34 GiB: about 6 s against 15 s on the measured host); the copies run at
// the same rate over either.  The threads that touch the pages first are bound to the CPUs of the NUMA node the GPU
// hangs off (when sysfs names one), so the arena lands next to this GPU's link and not on another socket whose
// memory the other GPUs' arenas already load.  Returns false when any step fails: the caller then falls back to
// cudaHostAlloc.
static bool map_arena(kvr_pool *p, size_t bytes) {
  // touching more memory than the host can give would invite the OOM killer; cudaHostAlloc fails politely instead
  unsigned long long avail_kb = 0;
  if (FILE *f = fopen("/proc/meminfo", "r")) {
    char line[256];
    while (fgets(line, sizeof line, f))
      if (sscanf(line, "MemAvailable: %llu kB", &avail_kb) == 1) break;
    fclose(f);
  }
  if (!avail_kb || (double)bytes > 0.9 * 1024.0 * (double)avail_kb) return false;
  const size_t huge = 2u << 20;
  const size_t len = align_up(bytes, huge) + huge;
  void *m = mmap(nullptr, len, PROT_READ | PROT_WRITE, MAP_PRIVATE | MAP_ANONYMOUS, -1, 0);
  if (m == MAP_FAILED) return false;
  char *base = reinterpret_cast<char *>(align_up(reinterpret_cast<uintptr_t>(m), huge));
  madvise(base, align_up(bytes, huge), MADV_HUGEPAGE);            // a hint: plain pages work too
  std::vector<int> cpus;
  char bus_id[32] = {0};
  int node = -1;
  if (cudaDeviceGetPCIBusId(bus_id, sizeof bus_id, p->device) == cudaSuccess) node = numa_lookup(nullptr, bus_id, &cpus);
  else cudaGetLastError();
  cpu_set_t set;
  CPU_ZERO(&set);
  bool bind = false;
  for (int c : cpus) if (c >= 0 && c < CPU_SETSIZE) { CPU_SET(c, &set); bind = true; }
  unsigned n_thr = std::thread::hardware_concurrency();
  n_thr = n_thr < 1 ? 1 : (n_thr > 8 ? 8 : n_thr);
  const size_t per = align_up((bytes + n_thr - 1) / n_thr, huge);
  std::vector<std::thread> touch;
  std::vector<int> bound(n_thr, 0);
  for (unsigned t = 0; t < n_thr; ++t)
    touch.emplace_back([=, &bound] {
      if (bind && sched_setaffinity(0, sizeof set, &set) == 0) bound[t] = 1;     // this thread only
      const size_t lo = (size_t)t * per, hi = lo + per < bytes ? lo + per : bytes;
      for (size_t o = lo; o < hi; o += 4096) base[o] = 0;
    });
  for (auto &t : touch) t.join();
  bool all_bound = bind;
  for (int b : bound) all_bound = all_bound && b;
  if (cudaHostRegister(base, bytes, cudaHostRegisterPortable | cudaHostRegisterMapped) != cudaSuccess) {
    cudaGetLastError();
    munmap(m, len);
    return false;
  }
  p->h_arena = base; p->arena_map = m; p->arena_map_len = len;
  p->numa_node = all_bound ? node : -1;
  return true;
}

kvr_status create_engine(kvr_pool *p) {
  const kvr_config &c = p->cfg;
  CU(cudaSetDevice(c.device));
  cudaDeviceProp prop;
  CU(cudaGetDeviceProperties(&prop, c.device));
  p->device = c.device;
  p->sm_count = prop.multiProcessorCount;
  if (c.route == KVR_ROUTE_DMA2D && (size_t)p->plane_stride > prop.memPitch)
    return fail(KVR_ERR_GEOMETRY, "strided-copy route: plane stride %lld exceeds the device's copy pitch limit %zu "
                "(use the block-major layout or another route)", p->plane_stride, prop.memPitch);
  const uint64_t pool_bytes = (uint64_t)p->NB * p->BS * p->bpt;
  if (c.device_pool) p->d_pool = (char *)c.device_pool;
  else {
    cudaError_t e = cudaMalloc((void **)&p->d_pool, pool_bytes);
    if (e != cudaSuccess) return fail(KVR_ERR_NOMEM, "cudaMalloc(pool, %llu): %s", (unsigned long long)pool_bytes, cudaGetErrorString(e));
    p->own_pool = true;
  }
  if (c.host_arena) p->h_arena = (char *)c.host_arena;
  else if (c.host_capacity_bytes) {
    if (!map_arena(p, c.host_capacity_bytes)) {
      cudaError_t e = cudaHostAlloc((void **)&p->h_arena, c.host_capacity_bytes, cudaHostAllocMapped);
      if (e != cudaSuccess) return fail(KVR_ERR_NOMEM, "cudaHostAlloc(arena, %llu): %s", (unsigned long long)c.host_capacity_bytes, cudaGetErrorString(e));
    }
    p->own_arena = true;
  }
  if (((uintptr_t)p->d_pool & 255) || ((uintptr_t)p->h_arena & 255))
    return fail(KVR_ERR_INVALID_ARG, "device_pool and host_arena must be 256-byte aligned");
  bool can_map = false;
  if (p->h_arena) {
    // the arena may be pinned host memory (the paper's host tier) or device memory: this GPU's, or a peer's that
    // this device can address.  Copies use cudaMemcpyDefault, so they follow the pointer wherever it lives.
    cudaPointerAttributes at{};
    if (c.host_arena && cudaPointerGetAttributes(&at, p->h_arena) == cudaSuccess && at.type == cudaMemoryTypeDevice) {
      p->arena_on_device = true;
      p->arena_dev = p->h_arena;
      can_map = true;
      if (at.device != c.device) {
        // a peer's memory: make it addressable from this device (the movers touch it with plain loads, stores and
        // single-CTA bulk copies only).  "Already enabled" is fine.
        cudaError_t pe = cudaDeviceEnablePeerAccess(at.device, 0);
        if (pe != cudaSuccess && pe != cudaErrorPeerAccessAlreadyEnabled) {
          cudaGetLastError();
          return fail(KVR_ERR_INVALID_ARG, "host_arena lives on device %d, which device %d cannot address: %s",
                      at.device, c.device, cudaGetErrorString(pe));
        }
        cudaGetLastError();
      }
    } else {
      cudaGetLastError();
      cudaError_t e = cudaHostGetDevicePointer((void **)&p->arena_dev, p->h_arena, 0);
      can_map = e == cudaSuccess;
      if (!can_map) { cudaGetLastError(); p->arena_dev = nullptr; }
      if (c.route == KVR_ROUTE_MAPPED && !can_map)
        return fail(KVR_ERR_INVALID_ARG, "host_arena is not mapped page-locked memory: %s", cudaGetErrorString(e));
    }
  }
  cudaStream_t *ss[4] = {&p->s_gather, &p->s_d2h, &p->s_h2d, &p->s_scatter};
  int lo = 0, hi = 0;
  CU(cudaDeviceGetStreamPriorityRange(&lo, &hi));
  for (int i = 0; i < 4; ++i) {
    if (c.streams[i]) { *ss[i] = static_cast<cudaStream_t>(c.streams[i]); continue; }
    CU(cudaStreamCreateWithPriority(ss[i], cudaStreamNonBlocking, hi));
    p->own_stream[i] = true;
  }
  for (int i = 0; i < 4; ++i)
    for (int j = i + 1; j < 4; ++j)
      if (*ss[i] == *ss[j]) return fail(KVR_ERR_INVALID_ARG, "the four streams must be distinct");
  p->route = c.route;
  if (p->route == KVR_ROUTE_AUTO || p->route == KVR_ROUTE_STAGED) {
    const int n = c.staging_slots;
    p->staging_total = (uint64_t)2 * n * c.chunk_bytes;
    if (c.device_staging) {
      if ((uintptr_t)c.device_staging & 255) return fail(KVR_ERR_INVALID_ARG, "device_staging must be 256-byte aligned");
      p->staging = (char *)c.device_staging;
    } else {
      cudaError_t e = cudaMalloc((void **)&p->staging, p->staging_total);
      if (e == cudaSuccess) p->own_staging = true;
      else {
        cudaGetLastError();
        p->staging = nullptr; p->staging_total = 0;
        if (p->route == KVR_ROUTE_STAGED || !can_map)
          return fail(KVR_ERR_NOMEM, "cudaMalloc(staging, %llu): %s", (unsigned long long)((uint64_t)2 * n * c.chunk_bytes), cudaGetErrorString(e));
        p->route = KVR_ROUTE_MAPPED;                 // auto: no staging memory to be had, the movers use the arena directly
      }
    }
    if (p->staging) {
      p->route = KVR_ROUTE_STAGED;
      p->slot_bytes = c.chunk_bytes;
      // How many of the ring's n slots one launch may cover.  While the link drains (or fills) the slots a launch
      // leaves free, the next launch has to run: with m slots per launch, (n - m) slots of link time must cover the
      // mover's time for m slots.  At full speed the movers are ~50 times faster than a PCIe Gen5 link (3 TB/s of
      // payload against 57 GB/s), which allows all slots but one; a grid capped with max_ctas is slower in
      // proportion (bulk mover: ~20 GB/s per CTA; warp mover: ~4 GB/s per CTA), and an arena in device memory is
      // a faster "link".  A margin of 1.5 covers launch latencies; a capped grid never takes more than half the ring
      // (whoever capped it runs other kernels beside the movers, which may slow them further).
      const int full_grid = c.kernel == KVR_KERNEL_BULK ? p->sm_count : 5 * p->sm_count;
      const int grid = (c.max_ctas > 0 && c.max_ctas < full_grid) ? c.max_ctas : full_grid;
      const double mover_gbs = 3000.0 * grid / full_grid;
      const double link_gbs = p->arena_on_device ? 800.0 : 57.0;
      int m = (int)((double)n * mover_gbs / (mover_gbs + 1.5 * link_gbs));
      if (grid < full_grid && m > n / 2) m = n / 2;     // a capped grid shares the SMs with somebody: plain double buffering
      p->launch_slots = m < 1 ? 1 : (m > n - 1 ? n - 1 : m);
      for (int dir = 0; dir < 2; ++dir) {
        Ring &r = dir ? p->in_ring : p->out_ring;
        r.base = p->staging + (size_t)dir * n * c.chunk_bytes;
        r.slots.resize(n);
        for (int i = 0; i < n; ++i) CU(cudaEventCreateWithFlags(&r.slots[i].freed, cudaEventDisableTiming));
      }
    }
  }
  CU(cudaHostAlloc((void **)&p->status_word, 64, cudaHostAllocMapped));
  *p->status_word = 0;
  if (c.kernel == KVR_KERNEL_BULK) {
    // about 192 KiB of shared memory per SM: 3 stages of up to 32 KiB per pipeline, more pipelines for smaller tiles
    // (measured on B200: 2 x 3 x 32 KiB for 32 KiB tiles, 8 x 3 x 8 KiB for 8 KiB tiles)
    int piece = p->tile_bytes < 32768 ? p->tile_bytes : 32768;
    int warps = (192 * 1024) / (3 * piece);
    warps = warps < 2 ? 2 : (warps > 8 ? 8 : warps);
    p->bulk = BulkShape{warps, 3, piece};
    if (c.bulk_warps || c.bulk_stages || c.bulk_piece_bytes) p->bulk = BulkShape{c.bulk_warps, c.bulk_stages, c.bulk_piece_bytes};
    cudaError_t e = bulk_configure(p->bulk);
    if (e != cudaSuccess) { cudaGetLastError(); return fail(KVR_ERR_INVALID_ARG, "bulk mover shape rejected: %s", cudaGetErrorString(e)); }
  }
  // everything a move needs exists before the first move: one descriptor buffer per move in flight, each large
  // enough for the block tables of the whole pool plus the segment records of a few thousand chunk pieces, and
  // a stock of events
  const size_t desc_cap = align_up((uint64_t)16 * p->NB + (256u << 10), 4096);
  p->descs.resize(c.max_moves_in_flight);
  for (auto &d : p->descs) if (kvr_status s = new_desc(desc_cap, &d)) return s;
  p->event_pool.reserve(4096);
  for (int i = 0; i < 512; ++i) {
    cudaEvent_t e;
    CU(cudaEventCreate(&e));
    p->event_pool.push_back(e);
  }
  p->pending_free.reserve(1024);
  return KVR_OK;
}

}  // namespace kvr
