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

// FIFO of free block ids in a fixed ring: blocks leave at the head and come
// back at the tail (released blocks rejoin at the eviction tail, Appendix A).
// Each entry carries the sequence number of the suspend whose gather may still
// be reading the block (0 = none), so a later writer can order itself after it.
class FreeQueue {
 public:
  void init(int32_t nb, const int32_t *order) {
    cap_ = nb; ring_.resize(nb); tag_.assign(nb, 0); in_queue_.assign(nb, 1);
    for (int32_t i = 0; i < nb; ++i) ring_[i] = order ? order[i] : i;
    head_ = 0; size_ = nb;
  }
  int64_t size() const { return size_; }
  // pop n ids from the head into out; returns the largest reader tag among them
  uint64_t pop(int32_t n, int32_t *out) {
    uint64_t tag = 0;
    for (int32_t i = 0; i < n; ++i) {
      int32_t b = ring_[head_];
      head_ = head_ + 1 == cap_ ? 0 : head_ + 1;
      out[i] = b; in_queue_[b] = 0;
      if (tag_[b] > tag) tag = tag_[b];
    }
    size_ -= n;
    return tag;
  }
  void push(const int32_t *ids, int32_t n, uint64_t reader_tag) {
    int64_t tail = head_ + size_;
    for (int32_t i = 0; i < n; ++i) {
      int64_t pos = tail + i; if (pos >= cap_) pos -= cap_;
      ring_[pos] = ids[i]; in_queue_[ids[i]] = 1; tag_[ids[i]] = reader_tag;
    }
    size_ += n;
  }
  bool is_free(int32_t b) const { return b >= 0 && b < cap_ && in_queue_[b]; }
  // remove the named ids (all known to be free and distinct), keeping the order of the rest
  uint64_t remove(const int32_t *ids, int32_t n) {
    uint64_t tag = 0;
    for (int32_t i = 0; i < n; ++i) { in_queue_[ids[i]] = 2; if (tag_[ids[i]] > tag) tag = tag_[ids[i]]; }
    std::vector<int32_t> keep; keep.reserve(size_);
    for (int64_t i = 0; i < size_; ++i) {
      int32_t b = at(i);
      if (in_queue_[b] == 2) in_queue_[b] = 0; else keep.push_back(b);
    }
    head_ = 0; size_ = (int64_t)keep.size();
    for (int64_t i = 0; i < size_; ++i) ring_[i] = keep[i];
    return tag;
  }
  int32_t at(int64_t i) const { int64_t pos = head_ + i; if (pos >= cap_) pos -= cap_; return ring_[pos]; }

 private:
  std::vector<int32_t> ring_;
  std::vector<uint64_t> tag_;
  std::vector<uint8_t> in_queue_;
  int64_t cap_ = 0, head_ = 0, size_ = 0;
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
  // len is a multiple of the granule and > 0
  bool alloc(uint64_t len, uint64_t *off) {
    for (auto it = holes_.begin(); it != holes_.end(); ++it) {
      if (it->second < len) continue;
      uint64_t o = it->first, rest = it->second - len;
      holes_.erase(it);
      if (rest) holes_[o + len] = rest;
      used_ += len; *off = o;
      return true;
    }
    return false;
  }
  void release(uint64_t off, uint64_t len) {
    used_ -= len;
    auto next = holes_.lower_bound(off);
    if (next != holes_.end() && off + len == next->first) { len += next->second; next = holes_.erase(next); }
    if (next != holes_.begin()) {
      auto prev = std::prev(next);
      if (prev->first + prev->second == off) { prev->second += len; return; }
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
  int32_t nb = 0;
  std::vector<int32_t> blocks;     // while ACTIVE / RETAINED
  uint64_t image_bytes = 0;
  uint64_t arena_off = 0, arena_len = 0;   // while HOST
  uint64_t pending_op = 0;         // sequence number of the move still in flight (0 = none)
  int32_t pending_kind = 0;        // KVR_SUSPENDING / KVR_RESUMING while pending_op != 0
  // timing of the last completed move
  bool has_latency = false;
  double host_ms = 0, device_ms = 0;
};

using RequestTable = std::unordered_map<uint64_t, Request>;

}  // namespace kvr
