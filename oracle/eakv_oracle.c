/*
 * Plain C restatement of the hot path's arithmetic -- TEST INFRASTRUCTURE ONLY (the timed CPU
 * baseline and a cross-check of the Python oracle).  It shares no code with the CUDA library and
 * the product never loads it.  Every function is the definition executed slowly:
 *
 *   oracle_hash_blocks   h_i = (h_{i-1} * B + token_i + 1) mod (2^61 - 1), key of block j = h after
 *                        its last token (Section 3.2: a key depends on the whole prefix; Section 4:
 *                        full chunks only).  One 128-bit product and one % per token.
 *   oracle_store / load  nested piece copies between the paged pool (2L arrays of
 *                        [blocks][piece_bytes]) and the slot-major tier [slots][2L][piece_bytes]
 *                        (Section 2; Appendix D: resident chunks are never copied again).
 *   oracle_tier_*        the LRU reference model of Appendix D under write-all or fixed admission
 *                        (Eq. 6 with p = 0 or p = 1): residents carry the time stamp of their last
 *                        reference, a hit refreshes it, an admitted miss takes a free slot (lowest
 *                        never-used first; an evicted slot is reused at once) after evicting the
 *                        resident with the smallest stamp when the tier is full.  Lookups and
 *                        victim searches are linear scans: slow, and correct by inspection.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define P61 ((((uint64_t)1) << 61) - 1)

int64_t oracle_hash_blocks(const int32_t* tokens, int64_t n_tokens, int32_t block_size, uint64_t parent,
                           uint64_t base, uint64_t* keys_out) {
    uint64_t h = parent % P61;
    int64_t nblk = 0;
    for (int64_t i = 0; i < n_tokens; ++i) {
        const unsigned __int128 t = (unsigned __int128)h * base + (uint64_t)((int64_t)tokens[i] + 1);
        h = (uint64_t)(t % P61);
        if ((i + 1) % block_size == 0) keys_out[nblk++] = h;
    }
    return nblk;
}

void oracle_store(uint8_t* const* pool, uint8_t* tier, int32_t pieces, int64_t piece_bytes,
                  const int32_t* block_table, const uint8_t* admit, const int32_t* slots, int64_t n) {
    for (int64_t j = 0; j < n; ++j) {
        if (admit && !admit[j]) continue;
        for (int32_t q = 0; q < pieces; ++q)
            memcpy(tier + ((int64_t)slots[j] * pieces + q) * piece_bytes,
                   pool[q] + (int64_t)block_table[j] * piece_bytes, (size_t)piece_bytes);
    }
}

void oracle_load(uint8_t* const* pool, const uint8_t* tier, int32_t pieces, int64_t piece_bytes,
                 const int32_t* slots, const int32_t* block_table, int64_t n) {
    for (int64_t j = 0; j < n; ++j)
        for (int32_t q = 0; q < pieces; ++q)
            memcpy(pool[q] + (int64_t)block_table[j] * piece_bytes,
                   tier + ((int64_t)slots[j] * pieces + q) * piece_bytes, (size_t)piece_bytes);
}

typedef struct {
    int64_t capacity, clock, next_fresh;
    int32_t policy, kappa;              /* policy 0: write-all, 1: fixed admission */
    uint64_t* key;                      /* by slot */
    int64_t* stamp;                     /* by slot: time of the last reference, -1 = free */
} oracle_tier;

oracle_tier* oracle_tier_new(int64_t capacity, int32_t policy, int32_t kappa) {
    oracle_tier* t = (oracle_tier*)calloc(1, sizeof(oracle_tier));
    t->capacity = capacity;
    t->policy = policy;
    t->kappa = kappa;
    t->key = (uint64_t*)calloc((size_t)capacity, sizeof(uint64_t));
    t->stamp = (int64_t*)malloc((size_t)capacity * sizeof(int64_t));
    for (int64_t s = 0; s < capacity; ++s) t->stamp[s] = -1;
    return t;
}

void oracle_tier_free(oracle_tier* t) {
    free(t->key);
    free(t->stamp);
    free(t);
}

static int64_t tier_find(const oracle_tier* t, uint64_t key) {
    for (int64_t s = 0; s < t->capacity; ++s)
        if (t->stamp[s] >= 0 && t->key[s] == key) return s;
    return -1;
}

/* leading run of resident keys, without touching recency */
int64_t oracle_tier_leading_run(const oracle_tier* t, const uint64_t* keys, int64_t n, int32_t* slots_out) {
    int64_t h = 0;
    for (; h < n; ++h) {
        const int64_t s = tier_find(t, keys[h]);
        if (s < 0) break;
        if (slots_out) slots_out[h] = (int32_t)s;
    }
    return h;
}

/* one request; returns -1 if it references more keys than the tier holds (nothing changes) */
int32_t oracle_tier_step(oracle_tier* t, const uint64_t* keys, int64_t n, uint8_t* hit, uint8_t* admit,
                         int32_t* slot) {
    if (n > t->capacity) return -1;
    const int64_t lead = oracle_tier_leading_run(t, keys, n, NULL);
    const int64_t u = n - lead;                                   /* new chunks of the request  */
    const int save = !(t->policy == 1 && u > t->kappa);           /* Eq. 6 with p = policy      */
    for (int64_t j = 0; j < n; ++j) {
        int64_t s = tier_find(t, keys[j]);
        hit[j] = s >= 0;
        admit[j] = 0;
        slot[j] = -1;
        if (s >= 0) {
            t->stamp[s] = t->clock++;
            slot[j] = (int32_t)s;
            continue;
        }
        if (!save) continue;
        if (t->next_fresh < t->capacity) {
            s = t->next_fresh++;                                  /* never-used slots, ascending */
        } else {
            s = 0;                                                /* evict the least recent      */
            for (int64_t v = 1; v < t->capacity; ++v)
                if (t->stamp[v] < t->stamp[s]) s = v;
        }
        t->key[s] = keys[j];
        t->stamp[s] = t->clock++;
        admit[j] = 1;
        slot[j] = (int32_t)s;
    }
    return save;
}
