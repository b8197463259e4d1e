// C ABI of the KV retention mover: bookkeeping + transfer engine.
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
#include <cuda_runtime.h>
#include <sched.h>
#include <sys/mman.h>

#include <algorithm>
#include <chrono>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "../../include/kvr.h"
#include "kvr_kernels.cuh"
#include "kvr_meta.hpp"
#include "kvr_numa.hpp"

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

// A CUDA runtime call on the move path.  Counted, and failed without being issued when a test armed the pool's
// failure hook for exactly this call (kvr_test_fail_nth).
#define CUP(p, call)                                                                          \
  do {                                                                                        \
    if (inject_cuda(p)) return fail(KVR_ERR_CUDA, "injected failure of %s", #call);          \
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
  std::vector<cudaEvent_t> aux;                     // per-chunk "ring filled" events
  std::vector<ReqDone> reqs;                        // request -> index of the chunk that completes it (-1: none)
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof;   // kernel brackets (KVR_PROFILE)
  int desc = -1;
  size_t stamp_off = 0; int n_stamps = 0;           // in-kernel time stamps inside the descriptor buffer (KVR_PROFILE)
  double host_ms = 0;
};

constexpr uint64_t kLeased = ~0ull;                 // DescBuf::busy of a buffer reserved by a call that has not enqueued yet
struct DescBuf { char *h = nullptr; char *d = nullptr; size_t cap = 0; uint64_t busy = 0; bool one_off = false; };
// A staging slot is handed back by an event.  Event operations cost the copy stream several microseconds each
// while the link is busy, so one recorded event usually stands for a run of slots: `owner` names the slot whose
// event object carries this slot's release, `seq` numbers the releases of a ring in the order they were recorded
// (all on one stream), so waiting for the largest `seq` among a set of slots covers the whole set.
struct Slot { cudaEvent_t freed = nullptr; bool used = false; uint64_t seq = 0; int owner = 0; };
struct Ring { char *base = nullptr; std::vector<Slot> slots; int next = 0; uint64_t seq = 0; };
struct PendingFree { uint64_t off, len, seq; };

// one request's part of a move
struct Item {
  uint64_t id;
  Request *r;
  const int32_t *blocks;   // the part of the table this move reads or writes (host copy)
  int32_t nb;              // its length
  int64_t n_tokens;        // tokens it covers
  uint64_t lin_off;        // offset of image byte 0 in the arena (or in the caller's device buffer)
  size_t bt_off;           // byte offset of its table inside the descriptor buffer
  int32_t batch_index;     // position in the caller's batch (per_req)
  int32_t prev_state;      // state to go back to if the move cannot be enqueued
};

struct CopyCmd { uint64_t lin_off; uint64_t ring_off; uint64_t vpos; uint64_t bytes; };
struct Chunk {
  int first_slot = 0, n_slots = 0;
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
  int route = KVR_ROUTE_STAGED;

  FreeQueue fq;
  Arena arena;
  RequestTable reqs;
  kvr_stats st{};

  // engine
  int device = 0, sm_count = 0;
  char *d_pool = nullptr; bool own_pool = false;
  char *h_arena = nullptr; bool own_arena = false;
  void *arena_map = nullptr; size_t arena_map_len = 0;   // own arena as a registered mapping (else cudaHostAlloc)
  int numa_node = -1;                     // node the own arena was faulted in on (-1: not placed)
  char *arena_dev = nullptr;              // device alias of the arena (mapped route)
  bool arena_on_device = false;           // the caller's arena is device memory (local or peer)
  cudaStream_t s_gather = nullptr, s_d2h = nullptr, s_h2d = nullptr, s_scatter = nullptr;
  bool own_stream[4] = {false, false, false, false};
  Ring out_ring, in_ring;
  char *staging = nullptr; bool own_staging = false;
  uint64_t slot_bytes = 0, staging_total = 0;
  int launch_slots = 1;                   // slots one mover launch may cover (at most all but one)
  int *status_word = nullptr;             // pinned + mapped: movers write it, the host reads it
  BulkShape bulk{4, 4, 8192};
  uint32_t call_flags = 0;                // flags of the call being served (set under the pool's lock)
  uint64_t copy_piece = 64ull << 20;      // largest single cudaMemcpyAsync of the staged route
  uint64_t suspend_single = 1ull << 30;   // a suspend up to this size is one launch (if it fits the ring)
  uint64_t resume_single = 256ull << 20;  // a resume up to this size is one launch
  std::vector<cudaEvent_t> event_pool;
  std::map<uint64_t, Op> ops;
  uint64_t next_seq = 1;
  std::vector<DescBuf> descs;
  std::vector<PendingFree> pending_free;
  std::mutex mu;                          // every entry point holds it: calls on one pool are serialised
  // host-made failures for tests: [0] CUDA calls, [1] host allocation points of the move path
  int64_t inject[2] = {0, 0}, points[2] = {0, 0};
};

namespace {

inline bool inject_cuda(kvr_pool *p) {
  ++p->points[KVR_FAIL_CUDA];
  return p->inject[KVR_FAIL_CUDA] > 0 && --p->inject[KVR_FAIL_CUDA] == 0;
}
// called right before the move path grows a host container
inline void alloc_point(kvr_pool *p) {
  ++p->points[KVR_FAIL_ALLOC];
  if (p->inject[KVR_FAIL_ALLOC] > 0 && --p->inject[KVR_FAIL_ALLOC] == 0) throw std::bad_alloc();
}

// ---- events, descriptors, op tracking ----------------------------------------------------

kvr_status get_event(kvr_pool *p, cudaEvent_t *out) {
  if (!p->event_pool.empty()) { *out = p->event_pool.back(); p->event_pool.pop_back(); return KVR_OK; }
  CUP(p, cudaEventCreate(out));
  return KVR_OK;
}
void put_event(kvr_pool *p, cudaEvent_t e) { if (e) p->event_pool.push_back(e); }

kvr_status new_desc(size_t cap, DescBuf *b) {
  b->cap = cap;
  CU(cudaHostAlloc((void **)&b->h, b->cap, cudaHostAllocDefault));
  cudaError_t e = cudaMalloc((void **)&b->d, b->cap);
  if (e != cudaSuccess) { cudaFreeHost(b->h); b->h = nullptr; return fail(KVR_ERR_NOMEM, "cudaMalloc(descriptors): %s", cudaGetErrorString(e)); }
  return KVR_OK;
}

void free_desc(DescBuf &b) {
  if (b.h) cudaFreeHost(b.h);
  if (b.d) cudaFree(b.d);
  b = DescBuf();
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

// byte offset, inside an item's image, of the first byte of tile q (q may equal the tile count)
inline uint64_t tile_off(const kvr_pool *p, const Item &it, long long q) {
  const long long plane = q / it.nb, b = q % it.nb;
  return ((uint64_t)plane * (uint64_t)it.n_tokens + (uint64_t)b * p->BS) * (uint64_t)p->row;
}

struct Plan {
  std::vector<Seg> segs;          // img pointers are final addresses
  std::vector<Chunk> chunks;
  std::vector<int> req_chunk;     // item -> last chunk that holds bytes of it (-1: none)
  int next_slot = 0;              // where the ring stands after the last chunk
};

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
uint64_t next_cap(const kvr_pool *p, uint64_t done, uint64_t total, bool resume, uint64_t big) {
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
    alloc_point(p);
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
  a.row_bytes = p->row; a.block_size = p->BS; a.num_blocks = p->NB; a.status = p->status_word; a.stamp = stamp;
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
void register_op(Op &op, std::vector<Item> &items, const std::vector<int> &req_chunk, int kind,
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
kvr_status enqueue_dma2d(kvr_pool *p, Op &op, std::vector<Item> &items, bool to_linear, uint64_t block_tag,
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
kvr_status enqueue_impl(kvr_pool *p, Op &op, int kind, std::vector<Item> &items, int route, char *lin_dev,
                        uint64_t block_tag, const std::vector<uint64_t> &arena_waits, Clock::time_point t_call,
                        int lease, uint64_t *out_seq) {
  const bool to_linear = (kind == OP_SUSPEND || kind == OP_EXPORT);
  kvr_status s = KVR_OK;
  if ((s = get_event(p, &op.start)) || (s = get_event(p, &op.read_done)) || (s = get_event(p, &op.done))) return s;
  alloc_point(p);
  op.reqs.resize(items.size());

  if (route == KVR_ROUTE_DMA2D) return enqueue_dma2d(p, op, items, to_linear, block_tag, arena_waits, t_call, out_seq);

  // plan with table addresses relative to the descriptor buffer, then size the buffer exactly:
  // [block tables][segments][stamps]
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
  size_t desc_bytes = n_stamps ? stamp_off + 16 * (size_t)n_stamps : seg_off + pl.segs.size() * sizeof(Seg);
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
      if ((s = launch(p, to_linear, segs_dev, ch, k, op, stamps_dev ? stamps_dev + 2 * ci : nullptr))) return s;
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
      if ((s = launch(p, true, segs_dev, ch, k, op, stamps_dev ? stamps_dev + 2 * ci : nullptr))) return s;
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
      if ((s = launch(p, false, segs_dev, ch, k, op, stamps_dev ? stamps_dev + 2 * ci : nullptr))) return s;
      if ((s = release(0, ch.n_slots, k))) return s;       // the scatter has read every slot of the chunk
      CUP(p, cudaEventRecord(cd, k));
    }
  }

  // read_done: the source of the move is no longer read.  done: the last byte has landed.
  cudaStream_t last = staged ? (to_linear ? c : k) : k;
  cudaStream_t reader = staged ? (to_linear ? k : c) : k;
  CUP(p, cudaEventRecord(op.read_done, reader));
  if (first != last) CUP(p, cudaStreamWaitEvent(last, op.read_done, 0));   // `done` must also cover the first stream (e.g. an empty move)
  if (n_stamps)      // the stamps come back with the move: `last` is ordered after every launch
    CUP(p, cudaMemcpyAsync(db.h + stamp_off, db.d + stamp_off, 16 * (size_t)n_stamps, cudaMemcpyDeviceToHost, last));
  CUP(p, cudaEventRecord(op.done, last));

  if (staged) ring->next = pl.next_slot;
  register_op(op, items, pl.req_chunk, kind, t_call, out_seq);
  return KVR_OK;
}

// A move could not be enqueued completely.  Part of it may already sit in the streams: wait for that work (it
// touches only staging memory, the arena range and the blocks the caller is about to take back), so that nothing of
// it is in flight when the bookkeeping is rolled back, then start the rings afresh.
void drain(kvr_pool *p) {
  for (cudaStream_t s : {p->s_gather, p->s_d2h, p->s_h2d, p->s_scatter}) if (s) cudaStreamSynchronize(s);
  cudaGetLastError();
  for (Ring *r : {&p->out_ring, &p->in_ring}) {
    for (auto &sl : r->slots) sl.used = false;
    r->next = 0;
  }
}

// after drain(): every event of the abandoned move has fired or was never recorded, so all of them can be reused
void abandon(kvr_pool *p, Op &op) {
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
