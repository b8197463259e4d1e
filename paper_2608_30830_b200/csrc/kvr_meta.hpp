// Host-side bookkeeping of the KV retention library: free queue of block ids,
// host arena, request table.  No CUDA in this file.
#pragma once
#include <cstdint>
#include <map>
#include <unordered_map>
#include <vector>

namespace kvr {

constexpr uint64_t kArenaGranule = 4096;

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// Free queue of block ids as an intrusive doubly linked list indexed by block id (Appendix A: pinning takes a
// context's blocks out of the doubly linked free queue in O(1), unpinning returns them to the eviction tail).
// Blocks leave at the head and come back at the tail, so the order is FIFO; a named block is unlinked in O(1).
// Next to the links every block carries
//   - a reference count: how many (request, position) pairs name it; it is in the queue iff the count is 0;
//   - the sequence number of the last move whose gather read it (0 = none), so a later writer can order itself
//     after that gather on the device.
class FreeQueue {
 public:
  void init(int32_t nb, const int32_t *order) {
    cap_ = nb;
    next_.assign(nb, -1); prev_.assign(nb, -1); tag_.assign(nb, 0); refs_.assign(nb, 0); mark_.assign(nb, 0);
    head_ = tail_ = -1; size_ = 0;
    for (int32_t i = 0; i < nb; ++i) link_tail(order ? order[i] : i);
  }
  int64_t size() const { return size_; }
  int32_t capacity() const { return (int32_t)cap_; }
  bool is_free(int32_t b) const { return b >= 0 && b < cap_ && refs_[b] == 0; }
  int32_t refs(int32_t b) const { return refs_[b]; }
  uint64_t tag(int32_t b) const { return tag_[b]; }

  // Take n ids from the head into out (one reference each); returns the largest reader tag among them.
  uint64_t pop(int32_t n, int32_t *out) {
    uint64_t tag = 0;
    for (int32_t i = 0; i < n; ++i) {
      const int32_t b = head_;
      unlink(b);
      refs_[b] = 1; out[i] = b;
      if (tag_[b] > tag) tag = tag_[b];
    }
    return tag;
  }
  // Undo a pop: the ids go back to the head, in their original order.
  void unpop(const int32_t *ids, int32_t n) {
    for (int32_t i = n - 1; i >= 0; --i) { refs_[ids[i]] = 0; link_after(ids[i], -1); }
  }

  // Take n named ids out of the queue (one reference each), keeping the order of the rest.  All must be free and
  // distinct: otherwise nothing changes, *bad names the offender and the call returns false.  prevs (n entries)
  // receives what unclaim() needs to put them back exactly where they were.
  bool claim(const int32_t *ids, int32_t n, int32_t *prevs, uint64_t *tag, int32_t *bad) {
    for (int32_t i = 0; i < n; ++i) {
      const int32_t b = ids[i];
      if (b < 0 || b >= cap_ || refs_[b] != 0 || mark_[b]) {
        for (int32_t j = 0; j < i; ++j) mark_[ids[j]] = 0;
        *bad = b;
        return false;
      }
      mark_[b] = 1;
    }
    uint64_t t = 0;
    for (int32_t i = 0; i < n; ++i) {
      const int32_t b = ids[i];
      mark_[b] = 0;
      prevs[i] = prev_[b];
      unlink(b);
      refs_[b] = 1;
      if (tag_[b] > t) t = tag_[b];
    }
    *tag = t;
    return true;
  }
  void unclaim(const int32_t *ids, const int32_t *prevs, int32_t n) {
    for (int32_t i = n - 1; i >= 0; --i) { refs_[ids[i]] = 0; link_after(ids[i], prevs[i]); }
  }

  void add_ref(int32_t b) { refs_[b] += 1; }
  // Drop one reference; the block joins the tail when the last one goes.  Returns true if it was freed.
  bool drop_ref(int32_t b) {
    if (--refs_[b] > 0) return false;
    link_tail(b);
    return true;
  }
  void note_reader(const int32_t *ids, int32_t n, uint64_t seq) {
    for (int32_t i = 0; i < n; ++i) if (tag_[ids[i]] < seq) tag_[ids[i]] = seq;
  }

  // iteration, head first: for (b = first(); b >= 0; b = after(b))
  int32_t first() const { return head_; }
  int32_t after(int32_t b) const { return next_[b]; }

 private:
  void unlink(int32_t b) {
    const int32_t p = prev_[b], n = next_[b];
    if (p >= 0) next_[p] = n; else head_ = n;
    if (n >= 0) prev_[n] = p; else tail_ = p;
    prev_[b] = next_[b] = -1;
    --size_;
  }
  void link_after(int32_t b, int32_t p) {          // p = -1: at the head
    const int32_t n = p >= 0 ? next_[p] : head_;
    prev_[b] = p; next_[b] = n;
    if (p >= 0) next_[p] = b; else head_ = b;
    if (n >= 0) prev_[n] = b; else tail_ = b;
    ++size_;
  }
  void link_tail(int32_t b) { link_after(b, tail_); }

  std::vector<int32_t> next_, prev_, refs_;
  std::vector<uint64_t> tag_;
  std::vector<uint8_t> mark_;
  int64_t cap_ = 0, size_ = 0;
  int32_t head_ = -1, tail_ = -1;
};

// Host tier as a map of free holes keyed by offset; allocation takes the first
// hole that is large enough, release merges with both neighbours.
class Arena {
 public:
  void init(uint64_t capacity) {
    capacity_ = capacity; used_ = 0; holes_.clear();
    uint64_t usable = capacity / kArenaGranule * kArenaGranule;
    if (usable) holes_[0] = usable;
  }
  // len is a multiple of the granule and > 0.  Never allocates: the hole's node is erased or re-keyed in place.
  bool alloc(uint64_t len, uint64_t *off) {
    for (auto it = holes_.begin(); it != holes_.end(); ++it) {
      if (it->second < len) continue;
      const uint64_t o = it->first, rest = it->second - len;
      if (rest) {
        auto node = holes_.extract(it);
        node.key() = o + len; node.mapped() = rest;
        holes_.insert(std::move(node));
      } else {
        holes_.erase(it);
      }
      used_ += len; *off = o;
      return true;
    }
    return false;
  }
  // Merges with both neighbours; allocates a node only when the range touches neither.
  void release(uint64_t off, uint64_t len) {
    used_ -= len;
    auto next = holes_.lower_bound(off);
    if (next != holes_.begin()) {
      auto prev = std::prev(next);
      if (prev->first + prev->second == off) {
        prev->second += len;
        if (next != holes_.end() && prev->first + prev->second == next->first) { prev->second += next->second; holes_.erase(next); }
        return;
      }
    }
    if (next != holes_.end() && off + len == next->first) {
      auto node = holes_.extract(next);
      node.key() = off; node.mapped() += len;
      holes_.insert(std::move(node));
      return;
    }
    holes_[off] = len;
  }
  uint64_t capacity() const { return capacity_; }
  uint64_t used() const { return used_; }
  uint64_t largest_hole() const {
    uint64_t m = 0;
    for (auto &h : holes_) if (h.second > m) m = h.second;
    return m;
  }

 private:
  std::map<uint64_t, uint64_t> holes_;
  uint64_t capacity_ = 0, used_ = 0;
};

struct Request {
  int32_t state = 0;               // settled state (KVR_ACTIVE / RETAINED / HOST / EXPIRED)
  int64_t n_tokens = 0;
  int32_t nb = 0;                  // logical blocks, shared prefix included
  int32_t n_shared = 0;            // leading blocks that are a shared prefix: never moved, referenced in every state but EXPIRED
  std::vector<int32_t> blocks;     // ACTIVE / RETAINED: all nb ids; HOST: the n_shared prefix ids
  uint64_t image_bytes = 0;        // the private suffix: (n_tokens - n_shared * block_size) * bytes_per_token
  uint64_t arena_off = 0, arena_len = 0;   // while HOST
  uint64_t pending_op = 0;         // sequence number of the move still in flight (0 = none)
  int32_t pending_kind = 0;        // KVR_SUSPENDING / KVR_RESUMING while pending_op != 0
  // timing of the last completed move
  bool has_latency = false;
  double host_ms = 0, device_ms = 0;
};

using RequestTable = std::unordered_map<uint64_t, Request>;

}  // namespace kvr
