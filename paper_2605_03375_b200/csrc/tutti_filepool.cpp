// CPU-side GPU-file pool (paper Section 3.1, "Scalable GPU File Pool"): all object slots
// ("GPU files") exist from start-up; persisting a new KV chunk only takes a free slot and
// installs a hash mapping chunk key -> slot, so creation, reclamation and metadata work
// stay off the I/O path.  The index lives on the CPU because GPU hash tables insert and
// look up far slower (Section 2.4).  Slots are handed out in ascending id so that chunks
// stored one after another get neighbouring slots — which the descriptor build then
// coalesces — and slot s lives on device s mod n_devices (round-robin placement).
// Chunks whose slot is pinned (in a batch that is in flight) are never reclaimed; when no
// slot is free the least recently used unpinned chunk is evicted.
#include <cstdint>
#include <functional>
#include <new>
#include <queue>
#include <unordered_map>
#include <vector>

#include "../../include/tutti.h"

namespace {
struct Entry {
    uint64_t key;
    uint32_t pins;
    bool used;
    uint32_t lru_prev, lru_next;   // doubly linked list of used slots, most recent at tail
};
constexpr uint32_t NIL = 0xffffffffu;
}  // namespace

struct tutti_filepool {
    std::vector<Entry> slots;
    std::unordered_map<uint64_t, uint32_t> index;
    std::priority_queue<uint32_t, std::vector<uint32_t>, std::greater<uint32_t>> free_slots;
    uint32_t lru_head = NIL, lru_tail = NIL;
    uint64_t hits = 0, misses = 0, evictions = 0;

    void unlink(uint32_t s) {
        Entry &e = slots[s];
        if (e.lru_prev != NIL) slots[e.lru_prev].lru_next = e.lru_next; else lru_head = e.lru_next;
        if (e.lru_next != NIL) slots[e.lru_next].lru_prev = e.lru_prev; else lru_tail = e.lru_prev;
        e.lru_prev = e.lru_next = NIL;
    }
    void push_recent(uint32_t s) {
        Entry &e = slots[s];
        e.lru_prev = lru_tail;
        e.lru_next = NIL;
        if (lru_tail != NIL) slots[lru_tail].lru_next = s; else lru_head = s;
        lru_tail = s;
    }
    void touch(uint32_t s) { unlink(s); push_recent(s); }
};

extern "C" {

int tutti_filepool_create(uint64_t n_slots, tutti_filepool_t **out) {
    if (!out || n_slots == 0 || n_slots >= NIL) return TUTTI_EINVAL;
    tutti_filepool *p = new (std::nothrow) tutti_filepool();
    if (!p) return TUTTI_ENOMEM;
    p->slots.assign((size_t)n_slots, Entry{0, 0, false, NIL, NIL});
    std::vector<uint32_t> all((size_t)n_slots);
    for (uint32_t s = 0; s < (uint32_t)n_slots; ++s) all[s] = s;
    p->free_slots = decltype(p->free_slots)(std::greater<uint32_t>(), std::move(all));
    p->index.reserve((size_t)n_slots * 2);
    *out = p;
    return TUTTI_OK;
}

int tutti_filepool_destroy(tutti_filepool_t *p) {
    if (!p) return TUTTI_EINVAL;
    delete p;
    return TUTTI_OK;
}

int tutti_filepool_insert(tutti_filepool_t *p, uint64_t key, uint32_t *slot, int *was_present) {
    if (!p || !slot) return TUTTI_EINVAL;
    auto it = p->index.find(key);
    if (it != p->index.end()) {                 // the chunk is already stored: share its slot
        *slot = it->second;
        if (was_present) *was_present = 1;
        p->touch(it->second);
        return TUTTI_OK;
    }
    if (was_present) *was_present = 0;
    uint32_t s;
    if (!p->free_slots.empty()) {
        s = p->free_slots.top();
        p->free_slots.pop();
    } else {
        // reclaim the least recently used chunk that no batch in flight refers to
        s = p->lru_head;
        while (s != NIL && p->slots[s].pins) s = p->slots[s].lru_next;
        if (s == NIL) return TUTTI_EAGAIN;
        p->index.erase(p->slots[s].key);
        p->unlink(s);
        p->evictions++;
    }
    Entry &e = p->slots[s];
    e.key = key;
    e.pins = 0;
    e.used = true;
    p->index.emplace(key, s);
    p->push_recent(s);
    *slot = s;
    return TUTTI_OK;
}

int tutti_filepool_lookup(tutti_filepool_t *p, uint64_t key, uint32_t *slot) {
    if (!p || !slot) return TUTTI_EINVAL;
    auto it = p->index.find(key);
    if (it == p->index.end()) { p->misses++; return TUTTI_ENOENT; }
    p->hits++;
    p->touch(it->second);
    *slot = it->second;
    return TUTTI_OK;
}

int tutti_filepool_match_prefix(tutti_filepool_t *p, const uint64_t *keys, uint32_t n_keys,
                                uint32_t *slots, uint32_t *n_hit, int pin) {
    if (!p || (n_keys && (!keys || !slots)) || !n_hit) return TUTTI_EINVAL;
    uint32_t k = 0;
    for (; k < n_keys; ++k) {
        auto it = p->index.find(keys[k]);
        if (it == p->index.end()) break;        // a prefix: the first missing chunk ends the hit
        slots[k] = it->second;
        p->touch(it->second);
        if (pin) p->slots[it->second].pins++;
    }
    p->hits += k;
    if (k < n_keys) p->misses++;
    *n_hit = k;
    return TUTTI_OK;
}

int tutti_filepool_pin(tutti_filepool_t *p, uint32_t slot, int delta) {
    if (!p || slot >= p->slots.size() || !p->slots[slot].used) return TUTTI_EINVAL;
    Entry &e = p->slots[slot];
    if (delta < 0 && e.pins < (uint32_t)(-delta)) return TUTTI_EINVAL;
    e.pins = (uint32_t)((int64_t)e.pins + delta);
    return TUTTI_OK;
}

int tutti_filepool_remove(tutti_filepool_t *p, uint64_t key) {
    if (!p) return TUTTI_EINVAL;
    auto it = p->index.find(key);
    if (it == p->index.end()) return TUTTI_ENOENT;
    uint32_t s = it->second;
    if (p->slots[s].pins) return TUTTI_EAGAIN;
    p->index.erase(it);
    p->unlink(s);
    p->slots[s].used = false;
    p->free_slots.push(s);
    return TUTTI_OK;
}

int tutti_filepool_stats(const tutti_filepool_t *p, uint64_t *used, uint64_t *free_slots,
                         uint64_t *hits, uint64_t *misses, uint64_t *evictions) {
    if (!p) return TUTTI_EINVAL;
    if (used) *used = p->index.size();
    if (free_slots) *free_slots = p->free_slots.size();
    if (hits) *hits = p->hits;
    if (misses) *misses = p->misses;
    if (evictions) *evictions = p->evictions;
    return TUTTI_OK;
}

}  // extern "C"
