// Host-side sub-allocator over the caller's device arena.  First fit with coalescing; every
// block is 256-byte aligned.  The library never calls cudaMalloc for relation data: running
// out of arena is the typed RESOURCE_EXHAUSTED outcome (Section "GPU residency model").
#pragma once
#include <cstddef>
#include <cstdint>
#include <map>

namespace xlog {

class Arena {
 public:
  void init(void* base, size_t bytes) {
    base_ = reinterpret_cast<uintptr_t>(base);
    const uintptr_t aligned = (base_ + 255) & ~uintptr_t(255);
    const size_t lost = aligned - base_;
    base_ = aligned;
    bytes_ = bytes > lost ? (bytes - lost) & ~size_t(255) : 0;
    free_.clear(); used_.clear();
    if (bytes_) free_[0] = bytes_;
    in_use_ = peak_ = 0;
  }
  void* alloc(size_t n) {
    if (n == 0) n = 1;
    n = (n + 255) & ~size_t(255);
    for (auto it = free_.begin(); it != free_.end(); ++it) {
      if (it->second >= n) {
        const size_t off = it->first, sz = it->second;
        free_.erase(it);
        if (sz > n) free_[off + n] = sz - n;
        used_[off] = n;
        in_use_ += n;
        if (in_use_ > peak_) peak_ = in_use_;
        return reinterpret_cast<void*>(base_ + off);
      }
    }
    return nullptr;
  }
  void release(void* p) {
    if (!p) return;
    const size_t off = reinterpret_cast<uintptr_t>(p) - base_;
    auto u = used_.find(off);
    if (u == used_.end()) return;
    size_t sz = u->second;
    size_t start = off;
    used_.erase(u);
    in_use_ -= sz;
    auto next = free_.lower_bound(start);
    if (next != free_.end() && start + sz == next->first) { sz += next->second; next = free_.erase(next); }
    if (next != free_.begin()) {
      auto prev = std::prev(next);
      if (prev->first + prev->second == start) { start = prev->first; sz += prev->second; free_.erase(prev); }
    }
    free_[start] = sz;
  }
  size_t in_use() const { return in_use_; }
  size_t peak() const { return peak_; }
  void reset_peak() { peak_ = in_use_; }
  size_t capacity() const { return bytes_; }
  size_t largest_free() const {
    size_t m = 0;
    for (auto& f : free_) if (f.second > m) m = f.second;
    return m;
  }

 private:
  uintptr_t base_ = 0;
  size_t bytes_ = 0, in_use_ = 0, peak_ = 0;
  std::map<size_t, size_t> free_, used_;
};

}  // namespace xlog
