#include "control_plane.h"

namespace eakv {

KeyedLru::KeyedLru(int64_t capacity)
    : cap_(capacity), resident_(0), node_(capacity, Node{0, -1, -1}),
      state_(capacity, 0), pin_count_(capacity, 0), lru_(-1), mru_(-1) {
    free_.reserve(capacity);
    for (int64_t s = capacity - 1; s >= 0; --s) free_.push_back((int32_t)s);
    size_t n = 16;
    while (n < (size_t)capacity * 2 + 2) n <<= 1;
    table_.assign(n, Entry{0, 0});
    mask_ = n - 1;
}

int32_t KeyedLru::find(uint64_t key) const {
    const uint64_t h = hash(key);
    const uint32_t tag = (uint32_t)h;
    size_t i = (size_t)h & mask_;
    while (true) {
        const Entry e = table_[i];
        if (e.v == 0) return -1;
        if (e.tag == tag && node_[e.v - 1].key == key) return e.v - 1;
        i = (i + 1) & mask_;
    }
}

void KeyedLru::table_put(uint64_t key, int32_t slot) {
    const uint64_t h = hash(key);
    size_t i = (size_t)h & mask_;
    while (table_[i].v != 0) i = (i + 1) & mask_;
    table_[i] = Entry{(uint32_t)h, slot + 1};
}

// linear probing with backward-shift deletion
void KeyedLru::table_erase(uint64_t key) {
    const uint64_t hk = hash(key);
    const uint32_t tag = (uint32_t)hk;
    size_t i = (size_t)hk & mask_;
    while (true) {
        const Entry e = table_[i];
        if (e.v == 0) return;
        if (e.tag == tag && node_[e.v - 1].key == key) break;
        i = (i + 1) & mask_;
    }
    size_t hole = i;
    size_t j = (i + 1) & mask_;
    while (table_[j].v != 0) {
        const size_t h = (size_t)table_[j].tag & mask_;
        // can the entry at j move into the hole?  yes unless its home lies cyclically in (hole, j]
        bool stays = (hole <= j) ? (h > hole && h <= j) : (h > hole || h <= j);
        if (!stays) {
            table_[hole] = table_[j];
            hole = j;
        }
        j = (j + 1) & mask_;
    }
    table_[hole] = Entry{0, 0};
}

void KeyedLru::unlink(int32_t s) {
    int32_t p = node_[s].prev, n = node_[s].next;
    if (p >= 0) node_[p].next = n; else lru_ = n;
    if (n >= 0) node_[n].prev = p; else mru_ = p;
    node_[s].prev = node_[s].next = -1;
}

void KeyedLru::push_mru(int32_t s) {
    node_[s].prev = mru_;
    node_[s].next = -1;
    if (mru_ >= 0) node_[mru_].next = s; else lru_ = s;
    mru_ = s;
}

void KeyedLru::promote(int32_t s) {
    if (mru_ == s) return;
    unlink(s);
    push_mru(s);
}

int32_t KeyedLru::evict_lru(uint64_t* victim_key) {
    int32_t v = lru_;
    *victim_key = node_[v].key;
    table_erase(node_[v].key);
    unlink(v);
    state_[v] = 0;
    --resident_;
    free_.push_back(v);
    // the next victims are known: bring in the table line of the next one and the node of the one after
    if (lru_ >= 0) {
        const Node& n = node_[lru_];
        __builtin_prefetch(&table_[(size_t)hash(n.key) & mask_], 1);
        if (n.next >= 0) __builtin_prefetch(&node_[n.next], 1);
    }
    return v;
}

int32_t KeyedLru::insert(uint64_t key, bool* evicted, uint64_t* victim_key, int32_t* victim_slot) {
    *evicted = false;
    if (resident_ >= cap_ || free_.empty()) {
        *victim_slot = evict_lru(victim_key);
        *evicted = true;
    }
    int32_t s = free_.back();
    free_.pop_back();
    node_[s].key = key;
    state_[s] = 1;
    table_put(key, s);
    push_mru(s);
    ++resident_;
    return s;
}

void KeyedLru::pin(int32_t s) {
    if (pin_count_[s]++ == 0) {
        unlink(s);
        ++pinned_;
    }
}

void KeyedLru::unpin(int32_t s) {
    if (--pin_count_[s] == 0) {
        push_mru(s);
        --pinned_;
    }
}

int32_t KeyedLru::erase(uint64_t key) {
    const int32_t s = find(key);
    if (s < 0 || pin_count_[s] > 0) return -1;
    table_erase(key);
    unlink(s);
    state_[s] = 0;
    --resident_;
    free_.push_back(s);
    return s;
}

int32_t KeyedLru::take_unkeyed(bool* evicted, uint64_t* victim_key, int32_t* victim_slot) {
    *evicted = false;
    if (free_.empty()) {
        *victim_slot = evict_lru(victim_key);
        *evicted = true;
    }
    int32_t s = free_.back();
    free_.pop_back();
    state_[s] = 2;
    return s;
}

void KeyedLru::release_unkeyed(int32_t s) {
    state_[s] = 0;
    free_.push_back(s);
}

int64_t KeyedLru::export_order(uint64_t* keys, int32_t* slots, int64_t capacity) const {
    int64_t n = 0;
    for (int32_t s = lru_; s >= 0; s = node_[s].next, ++n) {
        if (n < capacity) {
            if (keys) keys[n] = node_[s].key;
            if (slots) slots[n] = s;
        }
    }
    return n;
}

bool KeyedLru::import_order(const uint64_t* keys, const int32_t* slots, int64_t n) {
    if (resident_ != 0 || (int64_t)free_.size() != cap_ || n < 0 || n > cap_) return false;
    int64_t done = 0;
    bool ok = true;
    for (; done < n; ++done) {
        const int32_t s = slots[done];
        if (s < 0 || s >= cap_ || state_[s] != 0 || find(keys[done]) >= 0) { ok = false; break; }
        node_[s].key = keys[done];
        state_[s] = 1;
        table_put(keys[done], s);
        push_mru(s);
        ++resident_;
    }
    if (!ok) {                     // undo: back to the empty tier
        for (int64_t i = 0; i < done; ++i) {
            const int32_t s = slots[i];
            table_erase(node_[s].key);
            unlink(s);
            state_[s] = 0;
        }
        resident_ = 0;
        return false;
    }
    free_.clear();
    for (int64_t s = cap_ - 1; s >= 0; --s)
        if (state_[s] == 0) free_.push_back((int32_t)s);
    return true;
}

Admission::Admission(int32_t policy, int32_t kappa_blocks, int32_t theta_percent,
                     int64_t window_ms, int32_t len_window, int32_t telemetry,
                     int64_t host_blocks, int32_t block_size, int64_t report_period_ms,
                     int64_t report_max_age_ms)
    : policy_(policy), kappa_(kappa_blocks), theta_percent_(theta_percent),
      telemetry_(telemetry), window_ms_(window_ms), host_blocks_(host_blocks),
      period_ms_(report_period_ms), max_age_ms_(report_max_age_ms),
      len_window_(len_window), block_size_(block_size), length_sum_(0) {}

void Admission::publish(int64_t now_ms, int64_t resident_now) {
    if (period_ms_ <= 0) return;
    const int64_t t = now_ms / period_ms_ * period_ms_;
    if (t < period_ms_ || t <= report_time_) return;
    // every earlier request came before t, so the tier as it stands is what that publication saw
    int64_t e = 0;
    for (const EvictRun& r : evict_runs_) e += (r.time > t - window_ms_ && r.time < t) ? r.count : 0;
    report_time_ = t;
    report_resident_ = resident_now;
    report_evicted_ = e;
}

bool Admission::pressure(int64_t agent, int64_t n_tokens, int64_t now_ms, int64_t resident_now) {
    agent_last_[agent] = now_ms;
    lengths_.push_back(n_tokens);
    length_sum_ += n_tokens;
    while ((int64_t)lengths_.size() > len_window_) {
        length_sum_ -= lengths_.front();
        lengths_.pop_front();
    }
    const int64_t lo = now_ms - window_ms_;
    while (!evict_runs_.empty() && evict_runs_.front().time <= lo) {
        evict_count_ -= evict_runs_.front().count;
        evict_runs_.pop_front();
    }
    if (policy_ == 0) return false;
    if (policy_ == 1) return true;
    int64_t active = 0;
    for (const auto& kv : agent_last_) active += kv.second > lo;
    // 128-bit products: lengths and capacities are far below 2^63 but their product need not be
    const __int128 lhs = (__int128)(active - 1) * (__int128)length_sum_;
    const __int128 rhs = (__int128)host_blocks_ * block_size_ * (__int128)lengths_.size();
    const bool estimate = lhs > rhs;
    if (!telemetry_) return estimate;
    if (period_ms_ > 0) {
        const bool fresh = report_time_ >= 0 && (max_age_ms_ <= 0 || now_ms - report_time_ <= max_age_ms_);
        if (!fresh) return estimate;
        return estimate && (__int128)100 * report_resident_ >= (__int128)theta_percent_ * host_blocks_ &&
               report_evicted_ > 0;
    }
    const bool full = (__int128)100 * resident_now >= (__int128)theta_percent_ * host_blocks_;
    const bool evicting = !evict_runs_.empty();
    return estimate && full && evicting;
}

int64_t Admission::export_state(int64_t* out, int64_t capacity) const {
    std::vector<int64_t> v;
    std::map<int64_t, int64_t> ordered(agent_last_.begin(), agent_last_.end());
    v.push_back((int64_t)ordered.size());
    for (const auto& kv : ordered) { v.push_back(kv.first); v.push_back(kv.second); }
    v.push_back((int64_t)lengths_.size());
    for (int64_t x : lengths_) v.push_back(x);
    v.push_back(evict_count_);
    for (const EvictRun& r : evict_runs_) v.insert(v.end(), (size_t)r.count, r.time);
    v.push_back(report_time_);
    v.push_back(report_resident_);
    v.push_back(report_evicted_);
    for (size_t i = 0; i < v.size() && (int64_t)i < capacity; ++i) out[i] = v[i];
    return (int64_t)v.size();
}

bool Admission::import_state(const int64_t* in, int64_t n) {
    int64_t i = 0;
    auto take = [&](int64_t* x) { if (i >= n) return false; *x = in[i++]; return true; };
    int64_t na = 0, nl = 0, ne = 0;
    std::unordered_map<int64_t, int64_t> agents;
    std::deque<int64_t> lengths;
    std::deque<EvictRun> evs;
    int64_t sum = 0;
    if (!take(&na) || na < 0 || na > (n - i) / 2) return false;
    for (int64_t k = 0; k < na; ++k) {
        int64_t a = 0, t = 0;
        if (!take(&a) || !take(&t)) return false;
        agents[a] = t;
    }
    if (!take(&nl) || nl < 0 || nl > len_window_ || nl > n - i) return false;
    for (int64_t k = 0; k < nl; ++k) {
        int64_t x = 0;
        if (!take(&x) || x < 0) return false;
        lengths.push_back(x);
        sum += x;
    }
    if (!take(&ne) || ne < 0 || ne != n - i - 3) return false;
    for (int64_t k = 0; k < ne; ++k) {
        int64_t x = 0;
        if (!take(&x)) return false;
        if (!evs.empty() && evs.back().time == x) evs.back().count += 1;
        else evs.push_back(EvictRun{x, 1});
    }
    int64_t rt = -1, rr = 0, re = 0;
    if (!take(&rt) || !take(&rr) || !take(&re) || rt < -1 || rr < 0 || re < 0) return false;
    report_time_ = rt;
    report_resident_ = rr;
    report_evicted_ = re;
    agent_last_.swap(agents);
    lengths_.swap(lengths);
    length_sum_ = sum;
    evict_runs_.swap(evs);
    evict_count_ = ne;
    return true;
}

}  // namespace eakv
