// C ABI of the KV retention mover: bookkeeping + transfer engine.
//
// Every batch call settles the bookkeeping at once (states, block tables, arena
// offsets: the same answers a synchronous implementation gives) and enqueues
// the byte movement on four streams:
//
//   suspend, staged route :  gather kernel -> staging slot   (s_gather)
//                            slot -> pinned arena, DMA        (s_d2h)
//   resume,  staged route :  pinned arena -> slot, DMA        (s_h2d)
//                            scatter kernel slot -> pool      (s_scatter)
//   mapped route          :  the kernel reads / writes the arena itself
//
// so a suspend and a resume use different streams and different staging rings
// and can overlap, one per link direction.  Hazards between calls are ordered
// on the device with events, not by blocking the caller:
//   - a block freed by a suspend carries that move's sequence number; whoever
//     takes the block next waits for that move's gather ("read_done");
//   - a host range freed by a resume is remembered with the move's sequence
//     number; a suspend that lands on it waits for the move's last read;
//   - a move on a request whose previous move is in flight waits for it.
#include <cuda_runtime.h>
#include <sys/mman.h>

#include <algorithm>
#include <chrono>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <thread>
#include <vector>

#include "../../include/kvr.h"
#include "kvr_kernels.cuh"
#include "kvr_meta.hpp"

using namespace kvr;

namespace kvr { void set_last_error(const char *msg); }

namespace {

thread_local std::string g_err;

kvr_status fail(kvr_status st, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return st;
}

}  // namespace

// lets the library's other source files report through kvr_last_error()
void kvr::set_last_error(const char *msg) { g_err = msg ? msg : ""; }

namespace {

#define CU(call)                                                                              \
  do {                                                                                        \
    cudaError_t e_ = (call);                                                                  \
    if (e_ != cudaSuccess)                                                                    \
      return fail(KVR_ERR_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
  } while (0)

using Clock = std::chrono::steady_clock;
double ms_since(Clock::time_point t0) { return std::chrono::duration<double, std::milli>(Clock::now() - t0).count(); }

kvr_status fold(kvr_status acc, kvr_status s) {
  if (s < 0) return (acc < 0 && acc < s) ? acc : s;
  if (acc < 0) return acc;
  return s > acc ? s : acc;
}

enum OpKind { OP_SUSPEND = 1, OP_RESUME = 2, OP_EXPORT = 3, OP_IMPORT = 4 };

struct ReqDone { uint64_t id; int chunk; };

struct Op {
  uint64_t seq = 0;
  int kind = 0;
  cudaEvent_t start = nullptr, read_done = nullptr, done = nullptr;
  std::vector<cudaEvent_t> chunk_done;              // one per chunk, in order
  std::vector<ReqDone> reqs;                        // request -> index of the chunk that completes it (-1: none)
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof;   // kernel brackets (KVR_PROFILE)
  int desc = -1;
  size_t stamp_off = 0; int n_stamps = 0;           // in-kernel time stamps inside the descriptor buffer (KVR_PROFILE)
  double host_ms = 0;
};

struct DescBuf { char *h = nullptr; char *d = nullptr; size_t cap = 0; uint64_t busy = 0; };
struct Slot { char *ptr = nullptr; cudaEvent_t filled = nullptr, freed = nullptr; bool used = false; };
struct Ring { std::vector<Slot> slots; int next = 0; };
struct PendingFree { uint64_t off, len, seq; };

// one request's part of a move
struct Item {
  uint64_t id;
  Request *r;
  const int32_t *blocks;   // host copy of the table used by this move
  int32_t nb;
  int64_t n_tokens;
  uint64_t lin_off;        // offset of image byte 0 in the arena (or in the caller's device buffer)
  size_t bt_off;           // byte offset of its table inside the descriptor buffer
};

struct CopyCmd { uint64_t lin_off; uint64_t slot_off; uint64_t bytes; };
struct Chunk {
  int slot = -1;
  size_t seg_begin = 0; int nsegs = 0;
  long long tiles = 0; uint64_t bytes = 0;
  std::vector<CopyCmd> copies;
};

}  // namespace

struct kvr_pool {
  kvr_config cfg{};
  bool meta_only = false, profile = false;
  uint64_t bpt = 0;
  int row = 0, tile_bytes = 0;
  long long plane_stride = 0, block_stride = 0;
  int32_t NB = 0, BS = 0, planes = 0;

  FreeQueue fq;
  Arena arena;
  RequestTable reqs;
  kvr_stats st{};

  // engine
  int device = 0, sm_count = 0;
  char *d_pool = nullptr; bool own_pool = false;
  char *h_arena = nullptr; bool own_arena = false;
  void *arena_map = nullptr; size_t arena_map_len = 0;   // own arena as a registered mapping (else cudaHostAlloc)
  char *arena_dev = nullptr;              // device alias of the arena (mapped route)
  bool arena_on_device = false;           // the caller's arena is device memory (local or peer)
  cudaStream_t s_gather = nullptr, s_d2h = nullptr, s_h2d = nullptr, s_scatter = nullptr;
  Ring out_ring, in_ring;
  char *staging = nullptr;
  int *status_word = nullptr;             // pinned + mapped: movers write it, the host reads it
  BulkShape bulk{4, 4, 8192};
  uint32_t call_flags = 0;                // flags of the call being served (set under the pool's lock)
  uint64_t copy_piece = 64ull << 20;      // largest single cudaMemcpyAsync of the staged route
  std::vector<cudaEvent_t> event_pool;
  std::map<uint64_t, Op> ops;
  uint64_t next_seq = 1;
  std::vector<DescBuf> descs;
  std::vector<PendingFree> pending_free;
  std::mutex mu;                          // every entry point holds it: calls on one pool are serialised
};

namespace {

// ---- events, descriptors, op tracking ----------------------------------------------------

kvr_status get_event(kvr_pool *p, cudaEvent_t *out) {
  if (!p->event_pool.empty()) { *out = p->event_pool.back(); p->event_pool.pop_back(); return KVR_OK; }
  CU(cudaEventCreate(out));
  return KVR_OK;
}
void put_event(kvr_pool *p, cudaEvent_t e) { if (e) p->event_pool.push_back(e); }

kvr_status get_desc(kvr_pool *p, size_t bytes, int *out) {
  for (size_t i = 0; i < p->descs.size(); ++i)
    if (!p->descs[i].busy && p->descs[i].cap >= bytes) { *out = (int)i; return KVR_OK; }
  DescBuf b;
  b.cap = 1 << 20;
  while (b.cap < bytes) b.cap <<= 1;
  CU(cudaHostAlloc((void **)&b.h, b.cap, cudaHostAllocDefault));
  cudaError_t e = cudaMalloc((void **)&b.d, b.cap);
  if (e != cudaSuccess) { cudaFreeHost(b.h); return fail(KVR_ERR_NOMEM, "cudaMalloc(descriptors): %s", cudaGetErrorString(e)); }
  p->descs.push_back(b);
  *out = (int)p->descs.size() - 1;
  return KVR_OK;
}

void retire(kvr_pool *p, Op &op) {
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
    const unsigned long long *st = reinterpret_cast<const unsigned long long *>(p->descs[op.desc].h + op.stamp_off);
    double ms = 0;
    for (int i = 0; i < op.n_stamps; ++i)
      if (st[2 * i + 1] > st[2 * i]) ms += (double)(st[2 * i + 1] - st[2 * i]) * 1e-6;
    if (op.kind == OP_SUSPEND || op.kind == OP_EXPORT) p->st.gather_kernel_ms += ms; else p->st.scatter_kernel_ms += ms;
  }
  for (auto e : op.chunk_done) put_event(p, e);
  put_event(p, op.start); put_event(p, op.read_done); put_event(p, op.done);
  if (op.desc >= 0) p->descs[op.desc].busy = 0;
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

// host-side bounded wait for one move (seq) or all (seq = 0)
kvr_status wait_ops(kvr_pool *p, uint64_t seq, int64_t timeout_ms, bool read_only = false) {
  if (p->meta_only) return KVR_OK;
  if (timeout_ms < 0) timeout_ms = 60000;
  auto t0 = Clock::now();
  for (unsigned spin = 0;; ++spin) {
    if (read_only && seq) {
      auto it = p->ops.find(seq);
      if (it == p->ops.end()) return KVR_OK;
      cudaError_t e = cudaEventQuery(it->second.read_done);
      if (e == cudaSuccess) return KVR_OK;
      if (e != cudaErrorNotReady) return fail(KVR_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
    } else {
      kvr_status s = poll(p);
      if (s != KVR_OK) return s;
      if (seq ? !p->ops.count(seq) : p->ops.empty()) break;
    }
    if (ms_since(t0) > (double)timeout_ms) return fail(KVR_ERR_TIMEOUT, "move still in flight after %lld ms", (long long)timeout_ms);
    if (spin > 2000) std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
  if (p->status_word && *(volatile int *)p->status_word != 0)
    return fail(KVR_ERR_CUDA, "a mover gave up on a bounded wait (status %d)", *(volatile int *)p->status_word);
  return KVR_OK;
}

// make stream s wait for a move's event, if the move is still in flight
kvr_status stream_after(kvr_pool *p, cudaStream_t s, uint64_t seq, bool read_only) {
  if (!seq) return KVR_OK;
  auto it = p->ops.find(seq);
  if (it == p->ops.end()) return KVR_OK;
  CU(cudaStreamWaitEvent(s, read_only ? it->second.read_done : it->second.done, 0));
  return KVR_OK;
}

// byte offset, inside a request's image, of the first byte of tile q (q may equal the tile count)
inline uint64_t tile_off(const kvr_pool *p, const Item &it, long long q) {
  const long long plane = q / it.nb, b = q % it.nb;
  return ((uint64_t)plane * (uint64_t)it.n_tokens + (uint64_t)b * p->BS) * (uint64_t)p->row;
}

struct Plan {
  std::vector<Seg> segs;          // img pointers are final addresses
  std::vector<Chunk> chunks;
  std::vector<int> req_chunk;     // item -> last chunk that holds bytes of it (-1: none)
};

// Size limit of the next chunk of a staged move, given how many bytes earlier chunks hold and how many the move
// has in all.  A chunk is never larger than everything before it (so sizes double from a small start: a suspend's
// first copy over the link starts after a few microseconds of gathering, and the first requests of a batched
// resume are complete after milliseconds), never larger than a slot, and, for a resume, never larger than half of
// what is left (so sizes halve towards the end and little scattering remains after the last copy).
uint64_t next_cap(const kvr_pool *p, uint64_t done, uint64_t total, bool ramp_down_too) {
  const uint64_t big = p->cfg.chunk_bytes;
  uint64_t small = 32ull << 20;
  if (small < (uint64_t)p->tile_bytes) small = align_up(p->tile_bytes, 4096);
  if (small > big) small = big;
  uint64_t cap = done > small ? done : small;
  if (ramp_down_too) {
    const uint64_t left = total > done ? total - done : 0;
    const uint64_t half = left / 2 > small ? left / 2 : small;
    if (half < cap) cap = half;
  }
  if (cap > big) cap = big;
  if (cap < (uint64_t)p->tile_bytes) cap = p->tile_bytes;
  return cap;
}

// Staged route: cut the concatenated images into chunks on tile boundaries; chunk k goes to slot
// (ring.next + k) mod slots and holds at most next_cap() bytes.
void plan_staged(kvr_pool *p, const std::vector<Item> &items, Ring &ring, bool ramp_down_too, const char *desc_dev, Plan &pl) {
  uint64_t total = 0;
  for (auto &it : items) total += (uint64_t)it.n_tokens * p->bpt;
  const int nslots = (int)ring.slots.size();
  Chunk cur;
  uint64_t fill = 0, done = 0, cap = 0;
  auto open = [&]() {
    cur = Chunk();
    cur.slot = (ring.next + (int)pl.chunks.size()) % nslots;
    cur.seg_begin = pl.segs.size();
    fill = 0;
    cap = next_cap(p, done, total, ramp_down_too);
  };
  auto flush = [&]() {
    if (cur.nsegs) { cur.bytes = fill; done += fill; pl.chunks.push_back(cur); }
    open();
  };
  open();
  pl.req_chunk.assign(items.size(), -1);
  for (size_t i = 0; i < items.size(); ++i) {
    const Item &it = items[i];
    const long long T = (long long)p->planes * it.nb;
    long long q0 = 0;
    while (q0 < T) {
      const uint64_t base = tile_off(p, it, q0), room = cap - fill;
      long long lo = q0, hi = T;           // largest q1 with tile_off(q1) - base <= room
      while (lo < hi) {
        const long long mid = (lo + hi + 1) >> 1;
        const uint64_t end = mid == T ? (uint64_t)it.n_tokens * p->bpt : tile_off(p, it, mid);
        if (end - base <= room) lo = mid; else hi = mid - 1;
      }
      if (lo == q0 || cur.nsegs == kMaxSegs) { flush(); continue; }
      const long long q1 = lo;
      const uint64_t end = q1 == T ? (uint64_t)it.n_tokens * p->bpt : tile_off(p, it, q1);
      const uint64_t bytes = end - base;
      char *slot_ptr = ring.slots[cur.slot].ptr;
      Seg sg{};
      sg.bt = reinterpret_cast<const int32_t *>(desc_dev + it.bt_off);
      sg.img = slot_ptr + fill - base;
      sg.n_tokens = it.n_tokens; sg.tile_begin = q0; sg.tile_count = q1 - q0; sg.nb = it.nb;
      pl.segs.push_back(sg);
      cur.nsegs++; cur.tiles += q1 - q0;
      const uint64_t lin = it.lin_off + base;
      if (!cur.copies.empty() && cur.copies.back().lin_off + cur.copies.back().bytes == lin &&
          cur.copies.back().slot_off + cur.copies.back().bytes == fill)
        cur.copies.back().bytes += bytes;
      else
        cur.copies.push_back({lin, fill, bytes});
      fill += bytes;
      pl.req_chunk[i] = (int)pl.chunks.size();
      q0 = q1;
      if (cap - fill < (uint64_t)p->row) flush();
    }
    // low-latency resume: close the chunk where a request ends, so the request is complete (its scatter launched)
    // as soon as its own bytes have arrived instead of waiting for the rest of a slot
    if (ramp_down_too && (p->call_flags & KVR_LOW_LATENCY) && T > 0 && cur.nsegs) flush();
  }
  flush();
}

// Direct routes (mapped arena, export / import): one linear buffer, launches of up to kMaxSegs requests.
void plan_direct(kvr_pool *p, const std::vector<Item> &items, char *lin_base, const char *desc_dev, Plan &pl) {
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
    pl.segs.push_back(sg);
    cur.nsegs++; cur.tiles += T; cur.bytes += (uint64_t)it.n_tokens * p->bpt;
    pl.req_chunk[i] = (int)pl.chunks.size();
  }
  if (cur.nsegs) pl.chunks.push_back(cur);
}

kvr_status launch(kvr_pool *p, bool gather, const Seg *segs_dev, const Chunk &c, cudaStream_t s, Op &op,
                  unsigned long long *stamp) {
  MoveArgs a{};
  a.segs = segs_dev + c.seg_begin; a.nsegs = c.nsegs; a.total_tiles = c.tiles;
  a.pool = p->d_pool; a.plane_stride = p->plane_stride; a.block_stride = p->block_stride; a.tile_bytes = p->tile_bytes;
  a.row_bytes = p->row; a.block_size = p->BS; a.status = p->status_word; a.stamp = stamp;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (p->profile) {
    kvr_status s0 = get_event(p, &e0); if (s0) return s0;
    s0 = get_event(p, &e1); if (s0) return s0;
    CU(cudaEventRecord(e0, s));
  }
  cudaError_t e = p->cfg.kernel == KVR_KERNEL_BULK
                      ? launch_move_bulk(gather, a, p->bulk, p->cfg.max_ctas, p->sm_count, s)
                      : launch_move_warp(gather, a, p->cfg.max_ctas, p->sm_count, s);
  if (e != cudaSuccess) return fail(KVR_ERR_CUDA, "mover launch: %s", cudaGetErrorString(e));
  if (p->profile) { CU(cudaEventRecord(e1, s)); op.prof.push_back({e0, e1}); }
  if (gather) { p->st.gather_launches++; p->st.gather_bytes += c.bytes; }
  else { p->st.scatter_launches++; p->st.scatter_bytes += c.bytes; }
  return KVR_OK;
}

void register_op(kvr_pool *p, Op &op, std::vector<Item> &items, const std::vector<int> &req_chunk, int kind,
                 Clock::time_point t_call, uint64_t *out_seq) {
  op.host_ms = ms_since(t_call);
  for (size_t i = 0; i < items.size(); ++i) {
    op.reqs.push_back({items[i].id, req_chunk[i]});
    if (items[i].r) {
      items[i].r->pending_op = op.seq;
      items[i].r->pending_kind = kind == OP_SUSPEND ? KVR_SUSPENDING : kind == OP_RESUME ? KVR_RESUMING : 0;
      items[i].r->has_latency = false;
    }
  }
  *out_seq = op.seq;
  p->ops.emplace(op.seq, std::move(op));
}

// Strided-copy route: no kernel and no staging.  For every block, one cudaMemcpy2DAsync moves its 2L tiles
// (rows of `width` valid bytes, `plane_stride` apart in the pool, one image plane apart in the arena).
kvr_status enqueue_dma2d(kvr_pool *p, Op &op, std::vector<Item> &items, bool to_linear, uint64_t block_tag,
                         const std::vector<uint64_t> &arena_waits, Clock::time_point t_call, uint64_t *out_seq) {
  cudaStream_t c = to_linear ? p->s_d2h : p->s_h2d;
  kvr_status s;
  CU(cudaEventRecord(op.start, c));
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
        CU(cudaMemcpy2DAsync(img_ptr, img_pitch, pool_ptr, (size_t)p->plane_stride, width, (size_t)p->planes, cudaMemcpyDefault, c));
        p->st.d2h_copies++; p->st.d2h_bytes += width * p->planes;
      } else {
        CU(cudaMemcpy2DAsync(pool_ptr, (size_t)p->plane_stride, img_ptr, img_pitch, width, (size_t)p->planes, cudaMemcpyDefault, c));
        p->st.h2d_copies++; p->st.h2d_bytes += width * p->planes;
      }
    }
    cudaEvent_t cd;
    if ((s = get_event(p, &cd))) return s;
    CU(cudaEventRecord(cd, c));
    req_chunk[i] = (int)op.chunk_done.size();
    op.chunk_done.push_back(cd);
  }
  CU(cudaEventRecord(op.read_done, c));
  CU(cudaEventRecord(op.done, c));
  register_op(p, op, items, req_chunk, op.kind, t_call, out_seq);
  return KVR_OK;
}

// Build and upload the descriptors of a move, then enqueue it.  `to_linear` = gather direction.
// route: KVR_ROUTE_STAGED, KVR_ROUTE_MAPPED, or 0 for a caller-supplied device buffer (lin_dev).
kvr_status enqueue_impl(kvr_pool *p, Op &op, int kind, std::vector<Item> &items, int route, char *lin_dev,
                        uint64_t block_tag, const std::vector<uint64_t> &arena_waits, Clock::time_point t_call,
                        uint64_t *out_seq) {
  const bool to_linear = (kind == OP_SUSPEND || kind == OP_EXPORT);
  kvr_status s = KVR_OK;
  if ((s = get_event(p, &op.start)) || (s = get_event(p, &op.read_done)) || (s = get_event(p, &op.done))) return s;

  if (route == KVR_ROUTE_DMA2D) return enqueue_dma2d(p, op, items, to_linear, block_tag, arena_waits, t_call, out_seq);

  // plan with table addresses relative to the descriptor buffer, then size the buffer exactly:
  // [block tables][segments]
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
  const size_t stamp_off = align_up(seg_off + pl.segs.size() * sizeof(Seg), 64);
  const int n_stamps = p->profile ? (int)pl.chunks.size() : 0;
  const size_t desc_bytes = n_stamps ? stamp_off + 16 * (size_t)n_stamps : seg_off + pl.segs.size() * sizeof(Seg);
  if ((s = get_desc(p, desc_bytes ? desc_bytes : 64, &op.desc))) return s;
  DescBuf &db = p->descs[op.desc];
  for (int i = 0; i < n_stamps; ++i) {
    unsigned long long *st = reinterpret_cast<unsigned long long *>(db.h + stamp_off) + 2 * i;
    st[0] = ~0ull; st[1] = 0;
  }
  op.stamp_off = stamp_off; op.n_stamps = n_stamps;
  unsigned long long *stamps_dev = n_stamps ? reinterpret_cast<unsigned long long *>(db.d + stamp_off) : nullptr;
  for (auto &it : items) if (it.nb) memcpy(db.h + it.bt_off, it.blocks, (size_t)it.nb * 4);
  for (auto &sg : pl.segs) sg.bt = reinterpret_cast<const int32_t *>(db.d + reinterpret_cast<uintptr_t>(sg.bt));
  if (!pl.segs.empty()) memcpy(db.h + seg_off, pl.segs.data(), pl.segs.size() * sizeof(Seg));
  const Seg *segs_dev = reinterpret_cast<const Seg *>(db.d + seg_off);
  db.busy = op.seq;

  // streams: `k` runs the kernel, `c` runs the copies (staged route only)
  cudaStream_t k = to_linear ? p->s_gather : p->s_scatter;
  cudaStream_t c = to_linear ? p->s_d2h : p->s_h2d;
  const bool staged = route == KVR_ROUTE_STAGED;
  cudaStream_t first = (staged && !to_linear) ? c : k;    // stream of the first byte moved
  cudaStream_t host_side = staged ? c : k;                // stream that touches the arena

  CU(cudaEventRecord(op.start, first));
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

  if (desc_bytes) {
    CU(cudaMemcpyAsync(db.d, db.h, desc_bytes, cudaMemcpyHostToDevice, k));
    p->st.desc_bytes += desc_bytes;
  }

  // size of one link copy: 64 MiB, or more when the move is so large that 64 MiB pieces would put thousands of
  // entries into the copy stream (a full stream queue blocks the caller, and with it the next call's overlap)
  uint64_t piece = p->copy_piece;
  {
    uint64_t total = 0;
    for (auto &ch : pl.chunks) total += ch.bytes;
    const uint64_t floor_piece = align_up(total / 256 + 1, 1 << 20);
    if (piece < floor_piece) piece = floor_piece;
  }
  for (size_t ci = 0; ci < pl.chunks.size(); ++ci) {
    const Chunk &ch = pl.chunks[ci];
    cudaEvent_t cd;
    if ((s = get_event(p, &cd))) return s;
    op.chunk_done.push_back(cd);
    if (!staged) {
      if ((s = launch(p, to_linear, segs_dev, ch, k, op, stamps_dev ? stamps_dev + 2 * ci : nullptr))) return s;
      CU(cudaEventRecord(cd, k));
      continue;
    }
    Slot &sl = ring->slots[ch.slot];
    if (to_linear) {
      if (sl.used) CU(cudaStreamWaitEvent(k, sl.freed, 0));
      if ((s = launch(p, true, segs_dev, ch, k, op, stamps_dev ? stamps_dev + 2 * ci : nullptr))) return s;
      CU(cudaEventRecord(sl.filled, k));
      CU(cudaStreamWaitEvent(c, sl.filled, 0));
      // the copies go out in pieces: one very large cudaMemcpyAsync to pinned memory sustains less than the same
      // bytes in 64 MiB calls on some hosts (51.5 vs 56.3 GB/s measured), and never more
      for (auto &cp : ch.copies)
        for (uint64_t o = 0; o < cp.bytes; o += piece) {
          const uint64_t n = cp.bytes - o < piece ? cp.bytes - o : piece;
          CU(cudaMemcpyAsync(p->h_arena + cp.lin_off + o, sl.ptr + cp.slot_off + o, n, cudaMemcpyDefault, c));
          p->st.d2h_copies++; p->st.d2h_bytes += n;
        }
      CU(cudaEventRecord(sl.freed, c));
      CU(cudaEventRecord(cd, c));
    } else {
      if (sl.used) CU(cudaStreamWaitEvent(c, sl.freed, 0));
      for (auto &cp : ch.copies)
        for (uint64_t o = 0; o < cp.bytes; o += piece) {
          const uint64_t n = cp.bytes - o < piece ? cp.bytes - o : piece;
          CU(cudaMemcpyAsync(sl.ptr + cp.slot_off + o, p->h_arena + cp.lin_off + o, n, cudaMemcpyDefault, c));
          p->st.h2d_copies++; p->st.h2d_bytes += n;
        }
      CU(cudaEventRecord(sl.filled, c));
      CU(cudaStreamWaitEvent(k, sl.filled, 0));
      if ((s = launch(p, false, segs_dev, ch, k, op, stamps_dev ? stamps_dev + 2 * ci : nullptr))) return s;
      CU(cudaEventRecord(sl.freed, k));
      CU(cudaEventRecord(cd, k));
    }
    sl.used = true;
  }
  if (staged) ring->next = (ring->next + (int)pl.chunks.size()) % (int)ring->slots.size();

  // read_done: the source of the move is no longer read.  done: the last byte has landed.
  cudaStream_t last = staged ? (to_linear ? c : k) : k;
  cudaStream_t reader = staged ? (to_linear ? k : c) : k;
  if (first != last) {
    // both streams took part: `done` must also cover the first one (e.g. an empty move)
    CU(cudaEventRecord(op.read_done, reader));
    CU(cudaStreamWaitEvent(last, op.read_done, 0));
  } else {
    CU(cudaEventRecord(op.read_done, reader));
  }
  if (n_stamps)      // the stamps come back with the move: `last` is ordered after every launch
    CU(cudaMemcpyAsync(db.h + stamp_off, db.d + stamp_off, 16 * (size_t)n_stamps, cudaMemcpyDeviceToHost, last));
  CU(cudaEventRecord(op.done, last));

  register_op(p, op, items, pl.req_chunk, kind, t_call, out_seq);
  return KVR_OK;
}

// A move that could not be enqueued completely: give back what it took.  The events may already sit in a
// stream, so they are destroyed (legal while pending) rather than reused.
void abandon(kvr_pool *p, Op &op) {
  for (auto &pr : op.prof) { if (pr.first) cudaEventDestroy(pr.first); if (pr.second) cudaEventDestroy(pr.second); }
  for (auto e : op.chunk_done) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : {op.start, op.read_done, op.done}) if (e) cudaEventDestroy(e);
  if (op.desc >= 0) p->descs[op.desc].busy = 0;
}

kvr_status enqueue(kvr_pool *p, int kind, std::vector<Item> &items, int route, char *lin_dev, uint64_t block_tag,
                   const std::vector<uint64_t> &arena_waits, Clock::time_point t_call, uint64_t *out_seq) {
  if (kvr_status s = poll(p)) return s;
  Op op;
  op.seq = p->next_seq++;
  op.kind = kind;
  const kvr_status s = enqueue_impl(p, op, kind, items, route, lin_dev, block_tag, arena_waits, t_call, out_seq);
  if (s != KVR_OK) abandon(p, op);      // on success the move was handed to p->ops
  return s;
}

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

void free_blocks(kvr_pool *p, Request &r, uint64_t tag) {
  p->fq.push(r.blocks.data(), r.nb, tag);
  r.blocks.clear(); r.blocks.shrink_to_fit();
}

void free_host(kvr_pool *p, Request &r, uint64_t reader_seq) {
  if (r.arena_len) {
    p->arena.release(r.arena_off, r.arena_len);
    if (reader_seq) p->pending_free.push_back({r.arena_off, r.arena_len, reader_seq});
  }
  r.arena_off = r.arena_len = 0;
}

// a call that must see a request at rest first waits (bounded) for its move
kvr_status settle(kvr_pool *p, Request &r) {
  if (!r.pending_op) return KVR_OK;
  return wait_ops(p, r.pending_op, 60000);
}

void destroy_engine(kvr_pool *p) {
  for (auto &d : p->descs) { if (d.h) cudaFreeHost(d.h); if (d.d) cudaFree(d.d); }
  for (Ring *r : {&p->out_ring, &p->in_ring})
    for (auto &s : r->slots) { if (s.filled) cudaEventDestroy(s.filled); if (s.freed) cudaEventDestroy(s.freed); }
  for (auto e : p->event_pool) cudaEventDestroy(e);
  if (p->staging) cudaFree(p->staging);
  if (p->status_word) cudaFreeHost(p->status_word);
  for (cudaStream_t s : {p->s_gather, p->s_d2h, p->s_h2d, p->s_scatter}) if (s) cudaStreamDestroy(s);
  if (p->own_pool && p->d_pool) cudaFree(p->d_pool);
  if (p->own_arena && p->h_arena) {
    if (p->arena_map) { cudaHostUnregister(p->h_arena); munmap(p->arena_map, p->arena_map_len); }
    else cudaFreeHost(p->h_arena);
  }
}

// Page-locked arena of the library's own: an anonymous mapping backed by transparent huge pages where the host
// offers them, faulted in by several threads and then registered with CUDA.  Locking 2 MiB pages is several times
// quicker than cudaHostAlloc's 4 KiB pages (34 GiB: about 6 s against 15 s on the measured host); the copies run at
// the same rate over either.  Returns false when any step fails: the caller then falls back to cudaHostAlloc.
bool map_arena(kvr_pool *p, size_t bytes) {
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
  unsigned n_thr = std::thread::hardware_concurrency();
  n_thr = n_thr < 1 ? 1 : (n_thr > 8 ? 8 : n_thr);
  const size_t per = align_up((bytes + n_thr - 1) / n_thr, huge);
  std::vector<std::thread> touch;
  for (unsigned t = 0; t < n_thr; ++t)
    touch.emplace_back([=] {
      const size_t lo = (size_t)t * per, hi = lo + per < bytes ? lo + per : bytes;
      for (size_t o = lo; o < hi; o += 4096) base[o] = 0;
    });
  for (auto &t : touch) t.join();
  if (cudaHostRegister(base, bytes, cudaHostRegisterPortable | cudaHostRegisterMapped) != cudaSuccess) {
    cudaGetLastError();
    munmap(m, len);
    return false;
  }
  p->h_arena = base; p->arena_map = m; p->arena_map_len = len;
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
  if (p->h_arena) {
    // the arena may be pinned host memory (the paper's host tier) or device memory: this GPU's, or a peer's that
    // this device can address.  Copies use cudaMemcpyDefault, so they follow the pointer wherever it lives.
    cudaPointerAttributes at{};
    if (c.host_arena && cudaPointerGetAttributes(&at, p->h_arena) == cudaSuccess && at.type == cudaMemoryTypeDevice) {
      p->arena_on_device = true;
      p->arena_dev = p->h_arena;
      if (at.device != c.device) {
        // a peer's memory: make it addressable from this device (plain loads, stores and copies only -- the movers
        // use no multicast).  "Already enabled" is fine.
        cudaError_t pe = cudaDeviceEnablePeerAccess(at.device, 0);
        if (pe != cudaSuccess && pe != cudaErrorPeerAccessAlreadyEnabled) {
          cudaGetLastError();
          return fail(KVR_ERR_INVALID_ARG, "host_arena lives on device %d, which device %d cannot address: %s",
                      at.device, c.device, cudaGetErrorString(pe));
        }
        cudaGetLastError();
      }
    } else if (c.route == KVR_ROUTE_MAPPED) {
      cudaGetLastError();
      cudaError_t e = cudaHostGetDevicePointer((void **)&p->arena_dev, p->h_arena, 0);
      if (e != cudaSuccess) return fail(KVR_ERR_INVALID_ARG, "host_arena is not mapped page-locked memory: %s", cudaGetErrorString(e));
    }
  }
  int lo = 0, hi = 0;
  CU(cudaDeviceGetStreamPriorityRange(&lo, &hi));
  for (cudaStream_t *s : {&p->s_gather, &p->s_d2h, &p->s_h2d, &p->s_scatter})
    CU(cudaStreamCreateWithPriority(s, cudaStreamNonBlocking, hi));
  if (const char *env = getenv("KVR_COPY_PIECE_MIB")) {      // tuning knob for benchmarks
    const long v = atol(env);
    if (v >= 1 && v <= (1 << 20)) p->copy_piece = (uint64_t)v << 20;
  }
  if (c.route == KVR_ROUTE_STAGED) {
    const int n = c.staging_slots;
    cudaError_t e = cudaMalloc((void **)&p->staging, (size_t)2 * n * c.chunk_bytes);
    if (e != cudaSuccess) return fail(KVR_ERR_NOMEM, "cudaMalloc(staging): %s", cudaGetErrorString(e));
    for (int dir = 0; dir < 2; ++dir) {
      Ring &r = dir ? p->in_ring : p->out_ring;
      r.slots.resize(n);
      for (int i = 0; i < n; ++i) {
        r.slots[i].ptr = p->staging + ((size_t)dir * n + i) * c.chunk_bytes;
        CU(cudaEventCreateWithFlags(&r.slots[i].filled, cudaEventDisableTiming));
        CU(cudaEventCreateWithFlags(&r.slots[i].freed, cudaEventDisableTiming));
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
    if (const char *env = getenv("KVR_BULK_SHAPE")) {   // "warps,stages,piece_bytes": tuning knob for benchmarks
      int w, s, b;
      if (sscanf(env, "%d,%d,%d", &w, &s, &b) == 3) p->bulk = BulkShape{w, s, b};
    }
    cudaError_t e = bulk_configure(p->bulk);
    if (e != cudaSuccess) return fail(KVR_ERR_INVALID_ARG, "bulk mover shape rejected: %s", cudaGetErrorString(e));
  }
  return KVR_OK;
}

// shared body of the four bookkeeping-only outcomes and of the per-request loops
struct Batch {
  kvr_status acc = KVR_OK;
  kvr_status *per;
  int i = 0;
  void put(kvr_status s) { if (per) per[i] = s; acc = fold(acc, s); ++i; }
};

}  // namespace

// ---- C ABI -------------------------------------------------------------------------------

extern "C" {

const char *kvr_last_error(void) { return g_err.c_str(); }

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
  if (!p->cfg.chunk_bytes) p->cfg.chunk_bytes = 512ull << 20;
  if (!p->cfg.staging_slots) p->cfg.staging_slots = 2;
  if (!p->cfg.route) p->cfg.route = KVR_ROUTE_STAGED;
  if (!p->cfg.kernel) p->cfg.kernel = KVR_KERNEL_BULK;
  kvr_status bad = KVR_OK;
  if (p->cfg.route != KVR_ROUTE_STAGED && p->cfg.route != KVR_ROUTE_MAPPED && p->cfg.route != KVR_ROUTE_DMA2D) bad = fail(KVR_ERR_INVALID_ARG, "unknown route");
  else if (p->cfg.layout != KVR_LAYER_MAJOR && p->cfg.layout != KVR_BLOCK_MAJOR) bad = fail(KVR_ERR_INVALID_ARG, "unknown layout");
  else if (p->cfg.kernel != KVR_KERNEL_WARP && p->cfg.kernel != KVR_KERNEL_BULK) bad = fail(KVR_ERR_INVALID_ARG, "unknown kernel");
  else if (p->cfg.chunk_bytes % 4096 || p->cfg.chunk_bytes < tile) bad = fail(KVR_ERR_INVALID_ARG, "chunk_bytes must be a multiple of 4096 and hold one tile");
  else if (p->cfg.staging_slots < 2 || p->cfg.staging_slots > 64) bad = fail(KVR_ERR_INVALID_ARG, "staging_slots must be in [2, 64]");
  else if (p->cfg.max_ctas < 0) bad = fail(KVR_ERR_INVALID_ARG, "max_ctas < 0");
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
    s = wait_ops(p, 0, 60000);
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
  if (nb > p->fq.size()) { p->st.hbm_full_rejects++; return KVR_HBM_FULL; }
  Request &r = p->reqs[id];
  r = Request();
  r.state = KVR_ACTIVE; r.n_tokens = n_tokens; r.nb = (int32_t)nb;
  r.image_bytes = (uint64_t)n_tokens * p->bpt;
  r.blocks.resize(nb);
  const uint64_t tag = p->fq.pop((int32_t)nb, r.blocks.data());
  if (out_blocks && nb) memcpy(out_blocks, r.blocks.data(), nb * 4);
  // the caller will write these blocks from its own stream: let any gather still reading them finish
  if (tag && !p->meta_only) return wait_ops(p, tag, 60000, true);
  return KVR_OK;
}

kvr_status kvr_request_admit_into(kvr_pool *p, uint64_t id, int64_t n_tokens, const int32_t *blocks, int32_t nb) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n_tokens < 0 || nb < 0 || (nb > 0 && !blocks)) return fail(KVR_ERR_INVALID_ARG, "bad size or block list");
  if ((n_tokens + p->BS - 1) / p->BS != (int64_t)nb) return fail(KVR_ERR_INVALID_ARG, "nb must equal ceil(n_tokens / block_size)");
  auto it = p->reqs.find(id);
  if (it != p->reqs.end() && it->second.state != KVR_EXPIRED) return fail(KVR_ERR_BAD_STATE, "request exists");
  std::vector<uint8_t> named(p->NB, 0);
  for (int32_t i = 0; i < nb; ++i) {
    if (!p->fq.is_free(blocks[i]) || named[blocks[i]]) return fail(KVR_ERR_INVALID_ARG, "block %d is not free or named twice", blocks[i]);
    named[blocks[i]] = 1;
  }
  const uint64_t tag = p->fq.remove(blocks, nb);
  Request &r = p->reqs[id];
  r = Request();
  r.state = KVR_ACTIVE; r.n_tokens = n_tokens; r.nb = nb;
  r.image_bytes = (uint64_t)n_tokens * p->bpt;
  r.blocks.assign(blocks, blocks + nb);
  if (tag && !p->meta_only) return wait_ops(p, tag, 60000, true);     // a gather may still be reading these blocks
  return KVR_OK;
}

kvr_status kvr_request_release(kvr_pool *p, uint64_t id) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  auto it = p->reqs.find(id);
  if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
  Request &r = it->second;
  if (kvr_status s = settle(p, r)) return s;
  if (r.state == KVR_ACTIVE || r.state == KVR_RETAINED) free_blocks(p, r, 0);
  if (r.state == KVR_HOST) free_host(p, r, 0);
  p->reqs.erase(it);
  return KVR_OK;
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
    auto it = p->reqs.find(req[i]);
    if (it == p->reqs.end()) { b.put(KVR_ERR_UNKNOWN_REQUEST); continue; }
    Request &r = it->second;
    if (r.state == KVR_EXPIRED) { b.put(KVR_ERR_BAD_STATE); continue; }
    if (kvr_status s = settle(p, r)) { b.put(s); continue; }
    if (r.state == KVR_HOST) { p->st.bytes_expired_from_host += r.image_bytes; free_host(p, r, 0); }
    else free_blocks(p, r, 0);
    r.state = KVR_EXPIRED;
    p->st.expires++; p->st.recompute_marked++;
    b.put(KVR_OK);
  }
  return b.acc;
}

kvr_status kvr_suspend_to_host(kvr_pool *p, const uint64_t *req, int32_t n, uint32_t flags, kvr_status *per_req) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n < 0 || (n > 0 && !req)) return fail(KVR_ERR_INVALID_ARG, "bad request list");
  const auto t_call = Clock::now();
  if (!p->meta_only) { if (kvr_status s = poll(p)) return s; }
  Batch b{KVR_OK, per_req};
  std::vector<Item> items;
  std::vector<uint64_t> arena_waits;
  for (int32_t i = 0; i < n; ++i) {
    auto it = p->reqs.find(req[i]);
    if (it == p->reqs.end()) { b.put(KVR_ERR_UNKNOWN_REQUEST); continue; }
    Request &r = it->second;
    if (r.state != KVR_ACTIVE && r.state != KVR_RETAINED) { b.put(KVR_ERR_BAD_STATE); continue; }
    const uint64_t len = align_up(r.image_bytes, kArenaGranule);
    uint64_t off = 0;
    if (len && !p->arena.alloc(len, &off)) { p->st.host_full_rejects++; b.put(KVR_HOST_FULL); continue; }
    for (auto &pf : p->pending_free)
      if (len && pf.off < off + len && off < pf.off + pf.len) arena_waits.push_back(pf.seq);
    r.arena_off = off; r.arena_len = len;
    items.push_back({req[i], &r, r.blocks.data(), r.nb, r.n_tokens, off, 0});
    r.state = KVR_HOST;
    p->st.suspends++; p->st.bytes_suspended += r.image_bytes;
    b.put(KVR_OK);
  }
  uint64_t seq = 0;
  if (!p->meta_only && !items.empty()) {
    if (kvr_status s = enqueue(p, OP_SUSPEND, items, p->cfg.route, nullptr, 0, arena_waits, t_call, &seq)) return s;
  }
  // the move has copied the tables; now the ids join the free tail in request order, each in
  // logical block order, tagged with this move
  for (auto &it : items) free_blocks(p, *it.r, seq);
  if (seq && (flags & KVR_SYNC)) { if (kvr_status s = wait_ops(p, seq, 60000)) return s; }
  return b.acc;
}

static kvr_status resume_common(kvr_pool *p, std::vector<Item> &items, uint64_t block_tag, uint32_t flags,
                                Clock::time_point t_call) {
  uint64_t seq = 0;
  if (!p->meta_only && !items.empty()) {
    std::vector<uint64_t> none;
    p->call_flags = flags;
    const kvr_status s = enqueue(p, OP_RESUME, items, p->cfg.route, nullptr, block_tag, none, t_call, &seq);
    p->call_flags = 0;
    if (s) return s;
  }
  for (auto &it : items) free_host(p, *it.r, seq);
  if (seq && (flags & KVR_SYNC)) return wait_ops(p, seq, 60000);
  return KVR_OK;
}

kvr_status kvr_resume_from_host(kvr_pool *p, const uint64_t *req, int32_t n, uint32_t flags, kvr_status *per_req) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (n < 0 || (n > 0 && !req)) return fail(KVR_ERR_INVALID_ARG, "bad request list");
  const auto t_call = Clock::now();
  Batch b{KVR_OK, per_req};
  std::vector<Item> items;
  uint64_t block_tag = 0;
  for (int32_t i = 0; i < n; ++i) {
    auto it = p->reqs.find(req[i]);
    if (it == p->reqs.end()) { b.put(KVR_ERR_UNKNOWN_REQUEST); continue; }
    Request &r = it->second;
    if (r.state == KVR_RETAINED) { r.state = KVR_ACTIVE; p->st.resident_resumes++; b.put(KVR_RESIDENT); continue; }
    if (r.state == KVR_EXPIRED) { b.put(KVR_RECOMPUTE); continue; }
    if (r.state != KVR_HOST) { b.put(KVR_ERR_BAD_STATE); continue; }
    if (r.nb > p->fq.size()) { p->st.hbm_full_rejects++; b.put(KVR_HBM_FULL); continue; }
    r.blocks.resize(r.nb);
    const uint64_t tag = p->fq.pop(r.nb, r.blocks.data());
    if (tag > block_tag) block_tag = tag;
    items.push_back({req[i], &r, nullptr, r.nb, r.n_tokens, r.arena_off, 0});
    r.state = KVR_ACTIVE;
    p->st.resumes++; p->st.bytes_resumed += r.image_bytes;
    b.put(KVR_OK);
  }
  for (auto &it : items) it.blocks = it.r->blocks.data();
  if (kvr_status s = resume_common(p, items, block_tag, flags, t_call)) return s;
  return b.acc;
}

kvr_status kvr_resume_from_host_into(kvr_pool *p, uint64_t req, const int32_t *blocks, int32_t nb, uint32_t flags) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (nb < 0 || (nb > 0 && !blocks)) return fail(KVR_ERR_INVALID_ARG, "bad block list");
  const auto t_call = Clock::now();
  auto it = p->reqs.find(req);
  if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
  Request &r = it->second;
  if (r.state != KVR_HOST) return fail(KVR_ERR_BAD_STATE, "request is not on the host");
  if (nb != r.nb) return fail(KVR_ERR_INVALID_ARG, "request holds %d blocks, %d named", r.nb, nb);
  std::vector<uint8_t> named(p->NB, 0);
  for (int32_t i = 0; i < nb; ++i) {
    if (!p->fq.is_free(blocks[i]) || named[blocks[i]]) return fail(KVR_ERR_INVALID_ARG, "block %d is not free or named twice", blocks[i]);
    named[blocks[i]] = 1;
  }
  const uint64_t tag = p->fq.remove(blocks, nb);
  r.blocks.assign(blocks, blocks + nb);
  std::vector<Item> items{{req, &r, r.blocks.data(), r.nb, r.n_tokens, r.arena_off, 0}};
  r.state = KVR_ACTIVE;
  p->st.resumes++; p->st.bytes_resumed += r.image_bytes;
  return resume_common(p, items, tag, flags, t_call);
}

static kvr_status device_copy(kvr_pool *p, int kind, const uint64_t *req, int32_t n, char *dev, uint64_t capacity,
                              uint64_t *offsets, uint32_t flags) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (p->meta_only) return fail(KVR_ERR_BAD_STATE, "metadata-only pool moves no data");
  if (n < 0 || (n > 0 && !req) || !dev || ((uintptr_t)dev & 255)) return fail(KVR_ERR_INVALID_ARG, "bad request list or buffer (256-byte aligned device pointer)");
  const auto t_call = Clock::now();
  std::vector<Item> items;
  uint64_t cursor = 0;
  for (int32_t i = 0; i < n; ++i) {
    auto it = p->reqs.find(req[i]);
    if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
    Request &r = it->second;
    if (r.state != KVR_ACTIVE && r.state != KVR_RETAINED) return fail(KVR_ERR_BAD_STATE, "request holds no blocks");
    cursor = align_up(cursor, 256);
    if (offsets) offsets[i] = cursor;
    items.push_back({req[i], &r, r.blocks.data(), r.nb, r.n_tokens, cursor, 0});
    cursor += r.image_bytes;
  }
  if (cursor > capacity) return fail(KVR_ERR_INVALID_ARG, "buffer holds %llu bytes, %llu needed", (unsigned long long)capacity, (unsigned long long)cursor);
  uint64_t seq = 0;
  std::vector<uint64_t> none;
  if (!items.empty())
    if (kvr_status s = enqueue(p, kind, items, 0, dev, 0, none, t_call, &seq)) return s;
  if (seq && (flags & KVR_SYNC)) return wait_ops(p, seq, 60000);
  return KVR_OK;
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
  if (timeout_ms < 0) timeout_ms = 60000;
  const auto t0 = Clock::now();
  // the lock is taken per look, not for the whole wait, so other threads keep working on the pool meanwhile
  for (unsigned spin = 0;; ++spin) {
    {
      Enter enter(p);
      uint64_t seq = 0;
      if (req_or_all != KVR_ALL) {
        auto it = p->reqs.find(req_or_all);
        if (it == p->reqs.end()) return fail(KVR_ERR_UNKNOWN_REQUEST, "unknown request");
        seq = it->second.pending_op;
        if (!seq) return KVR_OK;
      }
      const kvr_status s = wait_ops(p, seq, 0);
      if (s != KVR_ERR_TIMEOUT) return s;
    }
    if (ms_since(t0) > (double)timeout_ms) return fail(KVR_ERR_TIMEOUT, "move still in flight after %lld ms", (long long)timeout_ms);
    if (spin > 2000) std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
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
  for (auto &kv : p->reqs) {
    const Request &r = kv.second;
    if (r.state == KVR_ACTIVE) { s.n_active++; s.blocks_active += r.nb; }
    else if (r.state == KVR_RETAINED) { s.n_retained++; s.blocks_pinned += r.nb; }
    else if (r.state == KVR_HOST) s.n_host++;
    else if (r.state == KVR_EXPIRED) s.n_expired++;
  }
  s.host_capacity = p->arena.capacity(); s.host_used = p->arena.used(); s.host_largest_hole = p->arena.largest_hole();
  s.ops_in_flight = (int64_t)p->ops.size();
  *out = s;
  return KVR_OK;
}

int64_t kvr_free_queue(kvr_pool *p, int32_t *out, int64_t cap) {
  if (!p) return -1;
  Enter enter(p);
  const int64_t n = p->fq.size();
  if (out) for (int64_t i = 0; i < n && i < cap; ++i) out[i] = p->fq.at(i);
  return n;
}

kvr_status kvr_selftest_bounded_wait(kvr_pool *p, int32_t leave_error_set) {
  if (kvr_status s = check_pool(p)) return s;
  Enter enter(p);
  if (p->meta_only) return fail(KVR_ERR_BAD_STATE, "metadata-only pool has no device side");
  if (kvr_status s = wait_ops(p, 0, 60000)) return s;
  cudaError_t e = launch_wait_limit_probe(p->status_word, 4096, p->s_gather);
  if (e != cudaSuccess) return fail(KVR_ERR_CUDA, "probe launch: %s", cudaGetErrorString(e));
  CU(cudaStreamSynchronize(p->s_gather));
  const int seen = *(volatile int *)p->status_word;
  if (!leave_error_set) *p->status_word = 0;
  if (seen != 2) return fail(KVR_ERR_CUDA, "the bounded wait did not run out (status word %d)", seen);
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
  if (kvr_status s = wait_ops(p, 0, 60000)) return s;
  if (p->arena.used() != 0) return fail(KVR_ERR_BAD_STATE, "the probe overwrites the arena: it must hold no image");
  if (bytes > p->arena.capacity()) bytes = p->arena.capacity() / 4096 * 4096;
  char *dev = nullptr;
  cudaError_t e = cudaMalloc((void **)&dev, bytes);
  if (e != cudaSuccess) return fail(KVR_ERR_NOMEM, "cudaMalloc(probe, %llu): %s", (unsigned long long)bytes, cudaGetErrorString(e));
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
  cudaFree(dev);
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
