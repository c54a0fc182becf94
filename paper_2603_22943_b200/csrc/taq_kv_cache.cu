// Host-side cache of K~/V~ blocks for the serving path: text keys/values depend on the prompt and the checkpoint
// only (Sec. III-B: "text keys/values"), so a request whose (checkpoint, prompt) pair was seen before skips the K/V
// projection, and the unconditional prompt of classifier-free guidance is one shared entry per checkpoint.  The
// cache owns no memory: it hands out fixed-size entries of a caller-owned device arena and never touches the device.
#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <unordered_map>
#include <vector>

#include "taq.h"

namespace {

struct Key {
    uint64_t checkpoint, prompt;
    bool operator==(const Key& o) const { return checkpoint == o.checkpoint && prompt == o.prompt; }
};
struct KeyHash {
    size_t operator()(const Key& k) const {
        uint64_t x = k.checkpoint * 0x9E3779B97F4A7C15ull ^ (k.prompt + 0x632BE59BD9B4E019ull + (k.checkpoint << 6) + (k.checkpoint >> 2));
        x ^= x >> 31;
        return (size_t)x;
    }
};
struct Slot {
    Key key{0, 0};
    bool valid = false;
    int pins = 0;
    uint64_t tick = 0;      // last use; smaller = older
};

}  // namespace

struct taq_kv_cache {
    uint8_t* arena = nullptr;
    size_t entry_bytes = 0;
    std::vector<Slot> slots;
    std::unordered_map<Key, int, KeyHash> index;
    uint64_t clock = 0;
    taq_kv_cache_stats stats{};
    std::mutex mu;
};

extern "C" {

uint64_t taq_hash_prompt(const int32_t* token_ids, int32_t n_tokens) {
    uint64_t h = 0xcbf29ce484222325ull;             // FNV-1a, 64 bit, over the little-endian bytes of the token ids
    for (int32_t i = 0; i < n_tokens; ++i) {
        uint32_t t = (uint32_t)token_ids[i];
        for (int b = 0; b < 4; ++b) {
            h ^= (t >> (8 * b)) & 0xFFu;
            h *= 0x100000001b3ull;
        }
    }
    return h;
}

taq_kv_cache* taq_kv_cache_create(void* arena_dev, size_t arena_bytes, size_t entry_bytes) {
    if (!arena_dev || entry_bytes == 0 || (entry_bytes & 127u) || (reinterpret_cast<uintptr_t>(arena_dev) & 127u)) return nullptr;
    const size_t n = arena_bytes / entry_bytes;
    if (n == 0 || n > (1u << 30)) return nullptr;
    taq_kv_cache* c = new (std::nothrow) taq_kv_cache;
    if (!c) return nullptr;
    c->arena = (uint8_t*)arena_dev;
    c->entry_bytes = entry_bytes;
    c->slots.resize(n);
    c->stats.capacity = (int64_t)n;
    return c;
}

void taq_kv_cache_destroy(taq_kv_cache* c) { delete c; }

taq_status taq_kv_cache_acquire(taq_kv_cache* c, uint64_t checkpoint, uint64_t prompt, void** entry_dev, int32_t* hit) {
    if (!c || !entry_dev || !hit) return TAQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(c->mu);
    const Key k{checkpoint, prompt};
    auto it = c->index.find(k);
    if (it != c->index.end()) {
        Slot& s = c->slots[it->second];
        ++s.pins;
        s.tick = ++c->clock;
        ++c->stats.hits;
        *entry_dev = c->arena + (size_t)it->second * c->entry_bytes;
        *hit = 1;
        return TAQ_OK;
    }
    int victim = -1;
    for (int i = 0; i < (int)c->slots.size(); ++i) {          // a free entry first, else the least recently used unpinned one
        const Slot& s = c->slots[i];
        if (!s.valid) { victim = i; break; }
        if (s.pins == 0 && (victim < 0 || s.tick < c->slots[victim].tick)) victim = i;
    }
    if (victim < 0) return TAQ_ERR_BUFFER_TOO_SMALL;          // every entry is in use by a request in flight
    Slot& s = c->slots[victim];
    if (s.valid) {
        c->index.erase(s.key);
        ++c->stats.evictions;
    } else {
        ++c->stats.used;
    }
    s.key = k;
    s.valid = true;
    s.pins = 1;
    s.tick = ++c->clock;
    c->index.emplace(k, victim);
    ++c->stats.misses;
    *entry_dev = c->arena + (size_t)victim * c->entry_bytes;
    *hit = 0;
    return TAQ_OK;
}

taq_status taq_kv_cache_release(taq_kv_cache* c, uint64_t checkpoint, uint64_t prompt) {
    if (!c) return TAQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(c->mu);
    auto it = c->index.find(Key{checkpoint, prompt});
    if (it == c->index.end() || c->slots[it->second].pins == 0) return TAQ_ERR_INVALID_ARG;
    --c->slots[it->second].pins;
    return TAQ_OK;
}

taq_status taq_kv_cache_drop_checkpoint(taq_kv_cache* c, uint64_t checkpoint) {
    if (!c) return TAQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(c->mu);
    for (Slot& s : c->slots)
        if (s.valid && s.key.checkpoint == checkpoint && s.pins > 0) return TAQ_ERR_INVALID_ARG;   // still in use
    for (Slot& s : c->slots)
        if (s.valid && s.key.checkpoint == checkpoint) {
            c->index.erase(s.key);
            s.valid = false;
            --c->stats.used;
        }
    return TAQ_OK;
}

taq_status taq_kv_cache_get_stats(taq_kv_cache* c, taq_kv_cache_stats* out) {
    if (!c || !out) return TAQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(c->mu);
    *out = c->stats;
    return TAQ_OK;
}

}  // extern "C"
