// Activation arena bookkeeping: where each d_i (and the per-segment gradient buffer) lives inside
// one slab, and the slab's high-water mark.  Pure host code; the device only ever sees offsets.
#include <algorithm>

#include "internal.h"

namespace ckpt {

int64_t Arena::stack_top() const {
    int64_t t = 0;
    for (const Block& b : live_) if (!b.top) t = std::max(t, b.off + b.size);
    return t;
}

int64_t Arena::top_floor() const {
    int64_t f = capacity_;
    for (const Block& b : live_) if (b.top) f = std::min(f, b.off);
    return f;
}

void Arena::account(int64_t id, int64_t off, int64_t size, bool top) {
    live_.push_back({id, off, size, top});
    live_bytes_ += size;
    high_water_ = std::max(high_water_, live_bytes_);
    // extent = bytes of address space in use: the stack from below plus the temporaries from above
    extent_ = std::max(extent_, stack_top() + (capacity_ - top_floor()));
    events.push_back({1, id, off, size});
}

int Arena::alloc_stack(int64_t id, int64_t size, int64_t* offset) {
    int64_t off = stack_top();
    if (off + size > top_floor()) {
        set_error("arena too small: tensor %lld (%lld bytes) at offset %lld does not fit below %lld",
                  (long long)id, (long long)size, (long long)off, (long long)top_floor());
        return CKPT_E_ARENA_OOM;
    }
    account(id, off, size, false);
    *offset = off;
    return CKPT_OK;
}

int Arena::alloc_top(int64_t id, int64_t size, int64_t* offset) {
    int64_t off = top_floor() - size;
    if (off < stack_top()) {
        set_error("arena too small: temporary %lld (%lld bytes) does not fit above %lld",
                  (long long)id, (long long)size, (long long)stack_top());
        return CKPT_E_ARENA_OOM;
    }
    account(id, off, size, true);
    *offset = off;
    return CKPT_OK;
}

int Arena::release(int64_t id) {
    for (size_t i = 0; i < live_.size(); ++i) {
        if (live_[i].id == id) {
            live_bytes_ -= live_[i].size;
            events.push_back({0, id, live_[i].off, live_[i].size});
            live_.erase(live_.begin() + i);
            return CKPT_OK;
        }
    }
    set_error("arena: tensor %lld released but not live", (long long)id);
    return CKPT_E_BAD_ARG;
}

bool Arena::is_live(int64_t id) const {
    for (const Block& b : live_) if (b.id == id) return true;
    return false;
}

int64_t Arena::offset_of(int64_t id) const {
    for (const Block& b : live_) if (b.id == id) return b.off;
    return -1;
}

}  // namespace ckpt
