// Residency policy of the tenants' weight blocks on the device (host code only, no CUDA calls).
//
// The paper (Sec. 3.3) argues that a worker caches model weights at each level of the memory hierarchy: models have
// a fixed footprint, so the time to bring one in over PCIe is predictable, and with a high enough hit ratio in GPU
// memory the PCIe link stops being the bottleneck.  This class is that cache's bookkeeping: a fixed arena of device
// bytes, a first-fit free list with coalescing, and least-recently-used eviction driven by a logical clock that the
// caller supplies (one tick per batch), so the policy can be tested with a made-up clock and no GPU.
#pragma once

#include <stddef.h>
#include <stdint.h>

#include <algorithm>
#include <map>
#include <vector>

namespace mt {

class WeightCache {
public:
    struct Entry {
        size_t off = 0, size = 0;
        uint64_t last_use = 0;
    };
    struct Stats {
        uint64_t hits = 0, misses = 0, evictions = 0, bytes_loaded = 0;
    };
    enum Result { kHit = 0, kLoaded = 1, kNoRoom = -1 };

    void reset(size_t capacity, size_t align = 1024) {
        capacity_ = capacity;
        align_ = align ? align : 1;
        free_.clear();
        if (capacity) free_[0] = capacity;
        live_.clear();
        stats_ = Stats();
        resident_bytes_ = 0;
    }
    size_t capacity() const { return capacity_; }
    size_t resident_bytes() const { return resident_bytes_; }
    const Stats& stats() const { return stats_; }
    void clear_stats() { stats_ = Stats(); }
    bool resident(int id) const { return live_.count(id) != 0; }
    const Entry* find(int id) const {
        auto it = live_.find(id);
        return it == live_.end() ? nullptr : &it->second;
    }

    // Make block `id` of `size` bytes resident at time `tick`.  A resident block is a hit (its clock is refreshed).
    // Otherwise room is made by evicting least-recently-used blocks whose last use is OLDER than `tick` - blocks
    // touched at `tick` itself belong to the batch being prepared and stay - and the ids evicted are appended to
    // *evicted (each with the time of its last use in *evicted_last_use, when given).  kNoRoom: the block does not
    // fit beside what the current tick holds (blocks evicted on the way stay evicted).
    Result acquire(int id, size_t size, uint64_t tick, size_t* off_out, std::vector<int>* evicted,
                   std::vector<uint64_t>* evicted_last_use = nullptr) {
        auto it = live_.find(id);
        if (it != live_.end()) {
            it->second.last_use = tick;
            if (off_out) *off_out = it->second.off;
            ++stats_.hits;
            return kHit;
        }
        const size_t need = round_up(size);
        if (need == 0 || need > capacity_) return kNoRoom;
        size_t off = 0;
        while (!take(need, &off)) {
            int victim = -1;                 // least recently used among the blocks not touched at this tick; ties: lowest id
            uint64_t oldest = 0;
            for (const auto& kv : live_) {
                const uint64_t u = kv.second.last_use;
                if (u >= tick) continue;
                if (victim < 0 || u < oldest || (u == oldest && kv.first < victim)) { victim = kv.first; oldest = u; }
            }
            if (victim < 0) return kNoRoom;
            if (evicted) evicted->push_back(victim);
            if (evicted_last_use) evicted_last_use->push_back(oldest);
            drop(victim);
            ++stats_.evictions;
        }
        Entry e;
        e.off = off; e.size = need; e.last_use = tick;
        live_[id] = e;
        resident_bytes_ += need;
        ++stats_.misses;
        stats_.bytes_loaded += size;
        if (off_out) *off_out = off;
        return kLoaded;
    }

    // Mark every resident block as used at `tick` (a batch whose tenant set the host cannot see).
    void touch_all(uint64_t tick) {
        for (auto& kv : live_) kv.second.last_use = tick;
    }

    // The model is withdrawn: its bytes return to the free list (no eviction is counted).
    void release(int id) {
        if (live_.count(id)) drop(id);
    }

    // Largest block that could be placed right now without evicting anything.
    size_t largest_free() const {
        size_t m = 0;
        for (const auto& kv : free_) m = std::max(m, kv.second);
        return m;
    }

private:
    size_t round_up(size_t v) const { return (v + align_ - 1) / align_ * align_; }

    bool take(size_t need, size_t* off) {       // first fit
        for (auto it = free_.begin(); it != free_.end(); ++it) {
            if (it->second < need) continue;
            *off = it->first;
            const size_t rest = it->second - need, start = it->first;
            free_.erase(it);
            if (rest) free_[start + need] = rest;
            return true;
        }
        return false;
    }

    void drop(int id) {
        const Entry e = live_[id];
        live_.erase(id);
        resident_bytes_ -= e.size;
        size_t off = e.off, size = e.size;
        auto next = free_.lower_bound(off);
        if (next != free_.end() && off + size == next->first) {     // merge with the free range behind
            size += next->second;
            next = free_.erase(next);
        }
        if (next != free_.begin()) {                                // merge with the free range in front
            auto prev = std::prev(next);
            if (prev->first + prev->second == off) {
                off = prev->first;
                size += prev->second;
                free_.erase(prev);
            }
        }
        free_[off] = size;
    }

    size_t capacity_ = 0, align_ = 1024, resident_bytes_ = 0;
    std::map<size_t, size_t> free_;        // offset -> length
    std::map<int, Entry> live_;
    Stats stats_;
};

}  // namespace mt
