// Host-side control plane: keyed LRU tiers and write admission.  Integer-only.
//
// KeyedLru implements the paper's LRU reference model (Appendix D): residents in recency
// order, hit -> most-recent end, admitted miss -> insert at the most-recent end after
// evicting the least-recent resident when full.  Storage is flat: an open-addressing
// table maps a 61-bit key to a slot (each entry carries 32 bits of the key's hash, so a probe
// reads the key array only on a tag match and a deletion never does); recency links live in
// arrays indexed by slot; free slots come from a stack that first yields 0, 1, 2, ... and reuses
// an evicted slot next.
#pragma once
#include <cstdint>
#include <deque>
#include <map>
#include <unordered_map>
#include <vector>

namespace eakv {

class KeyedLru {
public:
    explicit KeyedLru(int64_t capacity);

    int64_t capacity() const { return cap_; }
    int64_t resident() const { return resident_; }

    // slot of key or -1; does not change recency
    int32_t find(uint64_t key) const;
    // move a resident slot to the most-recent end
    void promote(int32_t slot);
    // Insert an absent key at the most-recent end.  When full, first evicts the
    // least-recent resident and reports it through (*victim_key, *victim_slot).
    // Returns the slot given to key.  *evicted is set to whether an eviction happened.
    int32_t insert(uint64_t key, bool* evicted, uint64_t* victim_key, int32_t* victim_slot);
    // Remove a resident key: its slot goes back on the free stack (it is the next one handed
    // out).  Returns the slot, or -1 when the key is not resident.
    int32_t erase(uint64_t key);
    // take an unkeyed slot (evicting the least-recent resident when none is free)
    int32_t take_unkeyed(bool* evicted, uint64_t* victim_key, int32_t* victim_slot);
    // give an unkeyed slot back to the free stack
    void release_unkeyed(int32_t slot);
    bool is_unkeyed_taken(int32_t slot) const { return state_[slot] == 2; }
    // Pinning (a running request holds the slot): a pinned resident leaves the recency order, so
    // it can be neither evicted nor promoted; when its last holder unpins it, it re-enters at the
    // most-recent end.  insert / take_unkeyed must not be called when nothing is free and every
    // resident is pinned (callers check evictable() + free_slots() first).
    void pin(int32_t slot);
    void unpin(int32_t slot);
    bool is_pinned(int32_t slot) const { return pin_count_[slot] > 0; }
    int64_t evictable() const { return resident_ - pinned_; }
    int64_t free_slots() const { return (int64_t)free_.size(); }
    // Hints for a caller that knows its keys ahead of the walk; they change nothing.  Call them in
    // this order a few references apart: the table line of a key; then the node of the slot its
    // home entry names; then that node's two neighbours in the recency order.
    void prefetch_table(uint64_t key) const { __builtin_prefetch(&table_[(size_t)hash(key) & mask_]); }
    void prefetch_node(uint64_t key) const {
        const Entry e = table_[(size_t)hash(key) & mask_];
        if (e.v) __builtin_prefetch(&node_[e.v - 1], 1);
    }
    void prefetch_neighbours(uint64_t key) const {
        const Entry e = table_[(size_t)hash(key) & mask_];
        if (!e.v) return;
        const Node& n = node_[e.v - 1];
        if (n.prev >= 0) __builtin_prefetch(&node_[n.prev], 1);
        if (n.next >= 0) __builtin_prefetch(&node_[n.next], 1);
    }
    // Residents in recency order, least recent first, into keys[]/slots[] (either may be NULL);
    // returns how many there are (at most `capacity` are written).
    int64_t export_order(uint64_t* keys, int32_t* slots, int64_t capacity) const;
    // Fill an EMPTY tier: entry i becomes resident at slots[i], later entries more recent.  The
    // free stack afterwards yields the unused slots in ascending order, exactly as if the entries
    // had been inserted by a run that never evicted.  False (and nothing changes) when the tier
    // is not empty or the input repeats a key or slot or leaves the range.
    bool import_order(const uint64_t* keys, const int32_t* slots, int64_t n);

private:
    struct Entry {
        uint32_t tag;                  // low 32 bits of the key's hash: the home position is tag & mask_
        int32_t v;                     // slot + 1, 0 = empty
    };
    void table_put(uint64_t key, int32_t slot);
    void table_erase(uint64_t key);
    static uint64_t hash(uint64_t x) {
        x ^= x >> 31;
        x *= 0x7fb5d329728ea185ull;
        x ^= x >> 27;
        x *= 0x81dadef4bc2dd44dull;
        x ^= x >> 33;
        return x;
    }
    struct Node {                      // by slot: key and recency links share a cache line
        uint64_t key;
        int32_t prev, next;            // -1 ends
    };
    void unlink(int32_t slot);
    void push_mru(int32_t slot);
    int32_t evict_lru(uint64_t* victim_key);

    int64_t cap_, resident_;
    std::vector<Node> node_;
    std::vector<uint8_t> state_;       // 0 free, 1 keyed resident, 2 unkeyed taken
    std::vector<int32_t> pin_count_;   // holders per slot
    int64_t pinned_ = 0;               // residents with at least one holder
    int32_t lru_, mru_;
    std::vector<int32_t> free_;        // stack
    std::vector<Entry> table_;         // at most half full
    size_t mask_;                      // table size - 1 (at most 2^32 - 1: capacities are below 2^31)
};

// Pressure signal of Eq. 10 over virtual time, all integers:
//   estimate  (A_t - 1) * sum(len) > K_H * b * count     (beta cancels, C_H = K_H b beta)
//   full      100 * resident >= theta_percent * K_H
//   evicting  evictions in (now - window, now] > 0
// With a report period the last two are read from the latest published report instead, if one
// exists and is not older than the maximum age; otherwise p_t is the working-set test by itself.
class Admission {
public:
    Admission(int32_t policy, int32_t kappa_blocks, int32_t theta_percent, int64_t window_ms,
              int32_t len_window, int32_t telemetry, int64_t host_blocks, int32_t block_size,
              int64_t report_period_ms = 0, int64_t report_max_age_ms = 0);
    // Published tier reports (report_period_ms = P > 0): call before a request at now_ms changes
    // the tier.  If a publication time P, 2P, ... has passed since the latest report, the tier as
    // it stands (resident_now chunks, evictions inside the window before that time) becomes the
    // report of floor(now / P) * P.
    void publish(int64_t now_ms, int64_t resident_now);
    // registers the request (agent activity, prompt length), expires old evictions and
    // returns p_t; call once per request before the walk
    bool pressure(int64_t agent, int64_t n_tokens, int64_t now_ms, int64_t resident_now);
    void note_eviction(int64_t now_ms) {
        ++evict_count_;
        if (!evict_runs_.empty() && evict_runs_.back().time == now_ms) evict_runs_.back().count += 1;
        else evict_runs_.push_back(EvictRun{now_ms, 1});
    }
    int32_t kappa() const { return kappa_; }
    // The windows as a flat list of int64: n_agents, (agent, last time) pairs in ascending agent
    // order, n_lengths, the prompt lengths oldest first, n_evictions, the eviction times oldest
    // first, then the latest published report (time or -1, resident chunks, evictions).  export_state returns the number of values (at most `capacity` are written);
    // import_state replaces the windows and returns false (nothing changed) on a malformed list.
    int64_t export_state(int64_t* out, int64_t capacity) const;
    bool import_state(const int64_t* in, int64_t n);

private:
    int32_t policy_, kappa_, theta_percent_, telemetry_;
    int64_t window_ms_, host_blocks_;
    int64_t period_ms_, max_age_ms_;
    int64_t report_time_ = -1, report_resident_ = 0, report_evicted_ = 0;   // latest report; time -1: none yet
    int32_t len_window_, block_size_;
    std::unordered_map<int64_t, int64_t> agent_last_;
    std::deque<int64_t> lengths_;
    int64_t length_sum_;
    struct EvictRun { int64_t time, count; };     // evictions of one request share its time
    std::deque<EvictRun> evict_runs_;             // oldest first
    int64_t evict_count_ = 0;                     // sum of the counts
};

}  // namespace eakv
