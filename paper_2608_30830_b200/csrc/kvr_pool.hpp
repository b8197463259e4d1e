// Internal declarations shared by the transfer engine (kvr_engine.cu) and the C ABI (kvr_lib.cu): the pool
// object, the engine's records and the few engine functions the entry points call.  Not part of the ABI.
#pragma once
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

namespace kvr {

// records the message kvr_last_error() returns on this thread and passes the status through
kvr_status fail(kvr_status st, const char *fmt, ...);
void set_last_error(const char *msg);
const char *last_error_text();

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
inline double ms_since(Clock::time_point t0) { return std::chrono::duration<double, std::milli>(Clock::now() - t0).count(); }

inline kvr_status fold(kvr_status acc, kvr_status s) {
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
  size_t stamp_off = 0; int n_stamps = 0;           // launch records inside the descriptor buffer whose stamps are read back (KVR_PROFILE)
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

// One per mover launch, inside the move's descriptor buffer: the kernel's work counter (uploaded as zero) and, under
// KVR_PROFILE, the earliest start and latest end any of its CTAs stamped (%globaltimer nanoseconds).
struct LaunchRec { unsigned long long first_start, last_end, work, pad; };

struct CopyCmd { uint64_t lin_off; uint64_t ring_off; uint64_t vpos; uint64_t bytes; };
struct Chunk {
  int first_slot = 0, n_slots = 0;
  size_t seg_begin = 0; int nsegs = 0;
  long long tiles = 0; uint64_t bytes = 0;
  std::vector<CopyCmd> copies;
};

}  // namespace kvr

struct kvr_pool {
  kvr_config cfg{};
  bool meta_only = false, profile = false;
  uint64_t bpt = 0;
  int row = 0, tile_bytes = 0;
  long long plane_stride = 0, block_stride = 0;
  int32_t NB = 0, BS = 0, planes = 0;
  int route = KVR_ROUTE_STAGED;

  kvr::FreeQueue fq;
  kvr::Arena arena;
  kvr::RequestTable reqs;
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
  kvr::Ring out_ring, in_ring;
  char *staging = nullptr; bool own_staging = false;
  uint64_t slot_bytes = 0, staging_total = 0;
  int launch_slots = 1;                   // slots one mover launch may cover (at most all but one)
  int *status_word = nullptr;             // pinned + mapped: movers write it, the host reads it
  kvr::BulkShape bulk{4, 4, 8192};
  uint32_t call_flags = 0;                // flags of the call being served (set under the pool's lock)
  uint64_t copy_piece = 64ull << 20;      // largest single cudaMemcpyAsync of the staged route
  uint64_t suspend_single = 1ull << 30;   // a suspend up to this size is one launch (if it fits the ring)
  uint64_t resume_single = 256ull << 20;  // a resume up to this size is one launch
  std::vector<cudaEvent_t> event_pool;
  std::map<uint64_t, kvr::Op> ops;
  uint64_t next_seq = 1;
  std::vector<kvr::DescBuf> descs;
  std::vector<kvr::PendingFree> pending_free;
  std::mutex mu;                          // every entry point holds it: calls on one pool are serialised
  // host-made failures for tests: [0] CUDA calls, [1] host allocation points of the move path
  int64_t inject[2] = {0, 0}, points[2] = {0, 0};
};

namespace kvr {

inline bool inject_cuda(kvr_pool *p) {
  ++p->points[KVR_FAIL_CUDA];
  return p->inject[KVR_FAIL_CUDA] > 0 && --p->inject[KVR_FAIL_CUDA] == 0;
}
// called right before the move path grows a host container
inline void alloc_point(kvr_pool *p) {
  ++p->points[KVR_FAIL_ALLOC];
  if (p->inject[KVR_FAIL_ALLOC] > 0 && --p->inject[KVR_FAIL_ALLOC] == 0) throw std::bad_alloc();
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

// ---- engine (kvr_engine.cu) ----------------------------------------------------------------
kvr_status create_engine(kvr_pool *p);
void destroy_engine(kvr_pool *p);
kvr_status get_event(kvr_pool *p, cudaEvent_t *out);
void put_event(kvr_pool *p, cudaEvent_t e);
// retires every move whose last event has fired; reports a status word the movers left behind
kvr_status poll(kvr_pool *p);
// KVR_OK when move `seq` (its gather only, if read_only) is over, KVR_PENDING while it runs
kvr_status look(kvr_pool *p, uint64_t seq, bool read_only);
// waits for a move with the pool's lock given up (other threads may enter meanwhile)
kvr_status wait_unlocked(kvr_pool *p, std::unique_lock<std::mutex> &lock, uint64_t seq, bool read_only, int64_t timeout_ms);
kvr_status wait_locked(kvr_pool *p, uint64_t seq, int64_t timeout_ms);
kvr_status stream_after(kvr_pool *p, cudaStream_t s, uint64_t seq, bool read_only);
void plan_staged(kvr_pool *p, const std::vector<Item> &items, Ring &ring, bool ramp_down_too, const char *desc_dev, Plan &pl);
// Queues the byte movement of one move.  On failure nothing of it is left in the streams and no record of it remains.
kvr_status enqueue(kvr_pool *p, int kind, std::vector<Item> &items, int route, char *lin_dev, uint64_t block_tag,
                   const std::vector<uint64_t> &arena_waits, Clock::time_point t_call, int lease, uint64_t *out_seq);

}  // namespace kvr
