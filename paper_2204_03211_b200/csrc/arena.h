// Offset allocator for one context's arena (host-side bookkeeping only: it
// hands out byte offsets; the device base pointer is added by the caller).
// First fit over an address-ordered free list with coalescing on release.
#pragma once

#include <cstddef>
#include <map>

namespace psb {

class Arena {
 public:
  static constexpr size_t kAlign = 256;
  static constexpr size_t kNone = ~(size_t)0;

  explicit Arena(size_t capacity = 0) { reset(capacity); }

  void reset(size_t capacity) {
    cap_ = capacity / kAlign * kAlign;
    used_ = 0;
    free_.clear();
    if (cap_) free_[0] = cap_;
  }

  static size_t round_up(size_t n) { return (n + kAlign - 1) / kAlign * kAlign; }

  // Returns the offset of a range of round_up(bytes) bytes, or kNone.
  size_t alloc(size_t bytes) {
    const size_t need = round_up(bytes ? bytes : 1);
    for (auto it = free_.begin(); it != free_.end(); ++it) {
      if (it->second >= need) {
        const size_t off = it->first, len = it->second;
        free_.erase(it);
        if (len > need) free_[off + need] = len - need;
        used_ += need;
        return off;
      }
    }
    return kNone;
  }

  void release(size_t off, size_t bytes) {
    size_t len = round_up(bytes ? bytes : 1);
    used_ -= len;
    auto next = free_.lower_bound(off);
    if (next != free_.begin()) {
      auto prev = std::prev(next);
      if (prev->first + prev->second == off) {
        off = prev->first;
        len += prev->second;
        free_.erase(prev);
      }
    }
    if (next != free_.end() && off + len == next->first) {
      len += next->second;
      free_.erase(next);
    }
    free_[off] = len;
  }

  size_t capacity() const { return cap_; }
  size_t used() const { return used_; }
  size_t largest_free() const {
    size_t m = 0;
    for (auto& kv : free_) m = kv.second > m ? kv.second : m;
    return m;
  }

 private:
  size_t cap_ = 0, used_ = 0;
  std::map<size_t, size_t> free_;   // offset -> length
};

}  // namespace psb
