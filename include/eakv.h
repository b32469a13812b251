/*
 * eakv -- paged-KV offload path for concurrent agents on one B200 (sm_100a).
 *
 * The data path that EfficientAgent's host tier drives: every agent turn the prompt's
 * token blocks get prefix-dependent keys, the longest cached prefix is located on the
 * GPU and in a host tier, the host-covered part is restored into fresh paged blocks,
 * and the turn's new blocks are written to the host tier under an LRU reference model
 * with write admission.
 *
 * Conventions
 *   - Every function returns an int status: EAKV_OK (0) or a negative EAKV_E_* code.
 *     Nothing throws or aborts; on a validation failure no kernel is launched and no
 *     state changes.  eakv_strerror() names a code; eakv_last_cuda_error() gives the
 *     CUDA error text behind the most recent EAKV_E_CUDA of a context.
 *   - "host" pointers are ordinary CPU memory (pageable is fine) and are fully consumed
 *     before the call returns.  "device" pointers must be dereferenceable by kernels of
 *     the context's GPU (device memory, or pinned host memory under unified addressing).
 *     The calls that pass a caller's token or key pointer to a kernel (eakv_hash_blocks,
 *     eakv_hash_blocks_batched, eakv_hash_blocks_static, eakv_turn_begin, eakv_request_begin,
 *     the capacity-model entry points) and eakv_create (pool, adopted tier) ask the runtime what
 *     the address is and return EAKV_E_INVAL for ordinary host memory instead of launching.
 *   - The caller owns every buffer it passes.  The context owns its tier memory (unless
 *     adopted, see eakv_config.tier_memory), staging buffers, argument rings and side
 *     streams.
 *   - cuda_stream is a cudaStream_t cast to void* (NULL = the legacy default stream).
 *     hash/store/load only enqueue work: results are valid once the stream has reached
 *     the point after the call.
 *   - A context is not thread-safe.  Two calls of the same kind (hash, store, load) on
 *     one context must be ordered with respect to each other (same stream, or an event
 *     between them): each kind has one set of scratch / staging buffers.  A store and a
 *     load may run concurrently on two streams.  Where they meet in a tier slot the library
 *     orders them itself: a store into a slot that a restore enqueued earlier (on another
 *     stream) still reads waits for that restore, and a restore of a slot that a store enqueued
 *     earlier still fills waits for that store.  The same holds for pool blocks the library
 *     itself overwrites: a restore into a block that a store enqueued earlier on another stream
 *     still reads waits for that store, and eakv_turn_begin / eakv_request_begin make
 *     cuda_stream wait for such stores of the blocks the turn is handed (so an engine that fills
 *     them behind cuda_stream is ordered too).  Any other write of the engine into a block that a
 *     store still reads is the caller's to order.
 *   - Layouts: the paged pool is 2L separate arrays, kv_base[2*l] = layer l's K and
 *     kv_base[2*l+1] = its V, each [gpu_blocks][block_size][kv_heads][head_dim] of
 *     elem_bytes-sized elements; one such [block_size][kv_heads][head_dim] slab is a
 *     "piece".  The tier is slot-major: [host_blocks * chunk_blocks][L][2][block_size][kv_heads][head_dim].
 *     piece bytes must be a multiple of 16 and all base pointers 16-byte aligned.
 */
#ifndef EAKV_H
#define EAKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define EAKV_OK           0
#define EAKV_E_INVAL     -1   /* NULL pointer, bad shape, misaligned base, duplicate destination */
#define EAKV_E_RANGE     -2   /* block id >= gpu_blocks or slot >= host_blocks (or negative) */
#define EAKV_E_CAPACITY  -3   /* request larger than a tier, scratch or output buffer */
#define EAKV_E_NOMEM     -4   /* host, pinned or device allocation failed */
#define EAKV_E_CUDA      -5   /* a CUDA runtime call failed; see eakv_last_cuda_error */
#define EAKV_E_TIMEOUT   -6   /* a bounded device-side wait gave up (bulk-copy path) */
#define EAKV_E_BUSY      -7   /* a running request's GPU blocks do not fit beside those the other running
                                 requests hold: nothing changed; retry after a request was released */

/* write admission (Section 4, Eq. 6): save(r) = not (p_t and u > kappa) */
#define EAKV_POLICY_WRITE_ALL          0   /* p_t = 0: plain offload                      */
#define EAKV_POLICY_FILTER_FIXED       1   /* p_t = 1: fixed write admission              */
#define EAKV_POLICY_FILTER_CONDITIONED 2   /* p_t = pressure signal of Appendix D, Eq. 10 */

/* how bytes cross the host link */
#define EAKV_LINK_ZERO_COPY 0   /* kernels read/write the mapped pinned tier directly          */
#define EAKV_LINK_STAGED    1   /* (default) gather to HBM staging + copy engine on a side stream,
                                   double-buffered against the next gather (and the mirror) */
#define EAKV_LINK_COPY_ENGINE 2 /* no kernel at all: one strided copy-engine transfer per block (rows =
                                   the block's pieces, pitch = the distance between piece arrays), issued on
                                   the caller's stream.  Needs the 2L piece arrays to sit at one constant
                                   pitch (one [2L][gpu_blocks][piece] allocation) that, like the bytes of
                                   one block, does not exceed the device's largest copy pitch
                                   (cudaDevAttrMaxPitch, 2 GiB - 1 on current parts: for instance at most
                                   131,071 blocks of 16-KiB pieces); eakv_create returns EAKV_E_INVAL
                                   otherwise.  Uses no SM while the engine's own kernels run */

/* where the tier lives */
#define EAKV_TIER_PINNED_HOST 0 /* the product configuration                                   */
#define EAKV_TIER_DEVICE      1 /* tier in HBM: on-device gather/scatter, for the HBM roofline;
                                   always copied directly (link_strategy is ignored)           */

/* which device code moves the bytes */
#define EAKV_COPY_VECTOR 0      /* 16-byte vector loads/stores, coalesced                       */
#define EAKV_COPY_BULK   1      /* 1-D bulk async copies through a shared-memory ring (default).
                                   copy_path selects the code for device-resident buffers (an
                                   HBM tier, the staging buffers); what moves a mapped host tier
                                   is selected by host_copy_path below                            */

/* which device code moves the bytes of a mapped host tier (EAKV_LINK_ZERO_COPY, and the scattered
 * calls that EAKV_LINK_STAGED sends directly) */
#define EAKV_HOST_COPY_VECTOR    0  /* 16-byte loads and stores over the link                          */
#define EAKV_HOST_COPY_BULK_LOAD 1  /* (default of eakv_config_init) restores: bulk async copies host ->
                                       shared memory -> pool; stores keep the vector kernel.  With both
                                       directions busy this moves 78 GB/s where two vector kernels move 73 */
#define EAKV_HOST_COPY_BULK_BOTH 2  /* both directions through the bulk-copy ring                      */

/* GPU-tier recency order of one request's blocks after eakv_gpu_tier_step (the GPU tier belongs
 * to the serving engine in the paper, Section 2; both orders are this library's model of it) */
#define EAKV_FREE_ASCENDING 0   /* as referenced: the prompt's first block is the request's least
                                   recent, so it is the first of them to be evicted              */
#define EAKV_FREE_REVERSE   1   /* tail first, the way a paged engine frees a sequence: the last
                                   block is evicted first and what survives is still a prefix     */

typedef struct eakv_ctx eakv_ctx;

typedef struct eakv_config {
    int32_t num_layers, kv_heads, head_dim, block_size, elem_bytes;
    int64_t gpu_blocks;            /* NB: blocks in each of the 2L paged arrays                 */
    int64_t host_blocks;           /* K_H = floor(C_H / (b * beta)): tier capacity in blocks
                                      (in chunks when chunk_blocks > 1)                          */
    int64_t gpu_index_blocks;      /* K_G: blocks the GPU-tier LRU hands out (<= gpu_blocks);
                                      0 = gpu_blocks                                             */
    void* const* kv_base;          /* host array of 2L device pointers (copied at create)       */
    uint64_t hash_base, hash_seed; /* B and S of the prefix hash; 0 = library defaults          */
    int32_t policy;                /* EAKV_POLICY_*                                              */
    int32_t kappa_blocks;          /* write threshold kappa, in tier units (blocks, or chunks)   */
    int32_t theta_percent;         /* occupancy threshold theta, in percent (paper: 95)          */
    int32_t len_window;            /* prompt-length window, in requests (paper: 256)             */
    int64_t window_ms;             /* activity / eviction window (paper: 60 s)                   */
    int32_t telemetry;             /* 1: the tier's report (occupancy, evictions) is read; 0: no
                                      report, p_t is the working-set test of Eq. 10 alone        */
    int32_t link_strategy;         /* EAKV_LINK_*                                                */
    int32_t tier_location;         /* EAKV_TIER_*                                                */
    int32_t copy_path;             /* EAKV_COPY_*                                                */
    int32_t copy_ctas;             /* CTAs of the copy kernels; 0 = auto (device buffers: the SM count
                                      times the kernel's resident CTAs; host tier: see host_*_ctas) */
    int64_t staging_bytes;         /* per staging buffer (two per direction); 0 = 256 MiB        */
    int64_t max_call_blocks;       /* entries per argument-ring slot; 0 = 16384                  */
    int64_t hash_scratch_blocks;   /* block partials the hash scratch holds; 0 = 1 << 20        */
    int64_t min_staged_run_bytes;  /* EAKV_LINK_STAGED: a call whose runs of consecutive slots
                                      average fewer bytes than this goes zero-copy instead (the
                                      copy engine's per-copy cost outweighs its edge on scattered
                                      single blocks); 0 = 3 MiB, negative = always stage         */
    int32_t control_plane_only;    /* 1: bookkeeping only (match, tier step, GPU-tier step): no
                                      CUDA call is made, kv_base may be NULL, no tier memory is
                                      allocated; hash/store/load return EAKV_E_INVAL            */
    int32_t chunk_blocks;          /* two granularities (the paper's 1,024-token host chunks over
                                      16-token GPU blocks): the host tier's unit is a chunk of
                                      this many consecutive blocks.  host_blocks then counts
                                      chunks, eakv_tier_step takes one key per chunk and counts
                                      u in chunks, and the tier memory holds host_blocks *
                                      chunk_blocks block-sized slots: chunk slot s covers block
                                      slots s*chunk_blocks .. (s+1)*chunk_blocks-1 for
                                      eakv_store / eakv_load.  0 or 1: one granularity           */
    void*   tier_memory;           /* NULL: the context allocates the tier.  Else adopt this
                                      buffer of host_blocks * chunk_blocks * block bytes (pinned host memory
                                      for TIER_PINNED_HOST, device memory for TIER_DEVICE);
                                      it must outlive the context                               */
    int32_t gpu_free_order;        /* EAKV_FREE_*: recency order a request leaves its blocks in
                                      within the GPU tier                                        */
    int32_t write_behind;          /* 1: eakv_turn_end enqueues the turn's host write on a stream of the
                                      context, after what precedes it on the caller's stream, and returns
                                      with the caller's stream free.  The library orders what must wait
                                      for that write: every later store, a load that reads a slot the
                                      write still fills, and a later turn whose new blocks reuse a GPU
                                      block the write still reads (the caller's stream is then made to
                                      wait at eakv_turn_begin).  Call eakv_sync
                                      before reading the tier on the host                              */
    int64_t telemetry_period_ms;   /* Appendix D, pressure signal and parameter table (report interval 1 s,
                                      a report counts as fresh for 5 s).  0: the occupancy and eviction
                                      terms of Eq. 10 are read from the tier itself at every request.
                                      P > 0: they are read from the latest published report.  Reports are
                                      published at the virtual times P, 2P, ... (now_ms of eakv_tier_step);
                                      the report of time t describes the tier as the requests before t
                                      left it: resident units, and the evictions with a time in
                                      (t - window_ms, t).  A request at now_ms reads the report of
                                      floor(now_ms / P) * P                                               */
    int64_t telemetry_max_age_ms;  /* a report older than this is not fresh (0: any age is).  Without a
                                      fresh report -- before the first publication, too -- p_t is the
                                      working-set test of Eq. 10 alone                                    */
    int32_t host_copy_path;        /* EAKV_HOST_COPY_*                                                    */
    int32_t host_load_ctas;        /* CTAs of a kernel that reads the mapped host tier; 0 = copy_ctas if
                                      set, else 96 for the bulk-copy ring and 64 for the vector kernel    */
    int32_t host_store_ctas;       /* CTAs of a kernel that writes it; 0 = likewise.  Restores are
                                      non-posted reads and stores posted writes, so with both directions
                                      busy they want different grids                                      */
    int32_t reserved0;
} eakv_config;

typedef struct eakv_stats {
    /* tier bookkeeping */
    int64_t requests, references, hits, admitted, declined, evicted;
    int64_t declined_requests, pressure_requests, resident;
    /* data plane */
    int64_t tokens_hashed, blocks_stored, blocks_loaded, bytes_stored, bytes_loaded;
    int64_t kernel_launches, memcpy_calls;
} eakv_stats;

typedef struct eakv_step_info {
    int64_t host_prefix_blocks;    /* H: leading blocks the host tier held before the step      */
    int64_t new_chunks;            /* u = floor(n/b) - floor(h/b)                               */
    int32_t pressure;              /* p_t                                                        */
    int32_t save;                  /* save(r)                                                    */
} eakv_step_info;

/* Fill *cfg with zeros and the paper's controller defaults (Appendix D, parameter table:
 * theta 0.95, 60 s windows, 256 lookups, kappa 8), write-all policy, the staged host-link
 * strategy and the bulk copy path. */
int eakv_config_init(eakv_config* cfg);

/* Create a context on the current CUDA device.  Allocates the tier (pinned + mapped, or
 * device), staging buffers, argument rings, hash scratch and two side streams.
 * Errors: EAKV_E_INVAL (bad shape/pointers), EAKV_E_NOMEM, EAKV_E_CUDA. */
int eakv_create(const eakv_config* cfg, eakv_ctx** out);

/* Wait for all work the context enqueued, then free everything it owns. */
int eakv_destroy(eakv_ctx* ctx);

/* Block keys (Section 3.2: a full chunk's key depends on its entire prefix; Section 4:
 * only full chunks).  h_{-1} = parent_hash, h_i = (h_{i-1} * B + token_i + 1) mod 2^61-1,
 * canonical in [0, p); key of block j = h after its last token; n_blocks = n_tokens /
 * block_size, a partial tail has no key.  Pass the context's seed (hash_seed) as
 * parent_hash for a fresh prompt, or block j-1's key with the tokens from j*block_size
 * on to resume at a block boundary.
 *   tokens_dev  device, int32[n_tokens], ids >= 0
 *   hashes_dev  device, uint64[n_tokens / block_size] (written)
 *   n_blocks_out host, may be NULL
 * Asynchronous on cuda_stream.  Errors: EAKV_E_INVAL, EAKV_E_CUDA. */
int eakv_hash_blocks(eakv_ctx* ctx, const int32_t* tokens_dev, int64_t n_tokens,
                     uint64_t parent_hash, uint64_t* hashes_dev, int64_t* n_blocks_out,
                     void* cuda_stream);

/* The same for many prompts in one call (one kernel launch; large batches with block size 16,
 * 32 or 64 take two: the token phase, then one scan CTA per prompt).  Prompt i is tokens_dev[offsets[i] ..
 * offsets[i+1]) and starts from parents[i] (NULL: the seed for all).  Keys are packed:
 * prompt i's keys start at block_offsets_out[i] = sum_{k<i} len_k / block_size.
 *   offsets_host       host, int64[n_prompts + 1], non-decreasing
 *   parents_host       host, uint64[n_prompts] or NULL
 *   block_offsets_out  host, int64[n_prompts + 1] (written) or NULL
 * Errors: EAKV_E_INVAL, EAKV_E_CAPACITY (more blocks than the hash scratch, or more
 * prompts than max_call_blocks), EAKV_E_CUDA. */
int eakv_hash_blocks_batched(eakv_ctx* ctx, const int32_t* tokens_dev,
                             const int64_t* offsets_host, int64_t n_prompts,
                             const uint64_t* parents_host, uint64_t* hashes_dev,
                             int64_t* block_offsets_out, void* cuda_stream);

/* Longest cached prefix (Section 2 "Exact-prefix reuse"; Appendix C "Prefix coverage
 * from a reference stream"): G = leading keys resident in the GPU index, H = leading keys
 * resident in the host tier; each walk stops at its first absent key.  The restore run is
 * blocks [G, H) when H > G.  Does not change recency.
 *   hashes_host       host, uint64[n_blocks]
 *   gpu_block_ids_out host, int32[>= G] or NULL;  host_slots_out host, int32[>= H] or NULL
 *                     (size them n_blocks) */
int eakv_match(const eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks,
               int64_t* gpu_prefix_blocks, int64_t* host_prefix_blocks,
               int32_t* gpu_block_ids_out, int32_t* host_slots_out);

/* One request against the host tier (Appendix D "Reference model" and "Recency order";
 * write rule Eq. 6 with the pressure signal Eq. 10).  References the keys in order: a
 * resident key hits and moves to the most-recent end; a miss is inserted at the
 * most-recent end (evicting the least-recent key when full) if the request is saved,
 * else declined.  The save decision is taken once, before the walk, from
 * u = n_blocks - H.  admit[j] = 1 exactly for inserted keys: those are the blocks to
 * pass to eakv_store with slot[j]; resident keys are never copied again (deduplication).
 *   hit_out, admit_out  host, uint8[n_blocks];  slot_out host, int32[n_blocks] (-1 = declined)
 *   evicted_keys_out / evicted_slots_out  host arrays of *n_evicted_inout entries or NULL;
 *   n_evicted_inout  in: capacity of those arrays, out: evictions of this step
 *                    (EAKV_E_CAPACITY, nothing changed, if capacity < n_blocks and non-NULL)
 *   info_out  host or NULL
 * Errors: EAKV_E_CAPACITY when n_blocks > host_blocks (nothing changes). */
int eakv_tier_step(eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks,
                   int64_t agent_id, int64_t n_tokens, int64_t now_ms,
                   uint8_t* hit_out, uint8_t* admit_out, int32_t* slot_out,
                   uint64_t* evicted_keys_out, int32_t* evicted_slots_out,
                   int64_t* n_evicted_inout, eakv_step_info* info_out);

/* A later lookup of a request whose write admission is already decided (Appendix D: the store or
 * skip choice of a request's first prefix lookup is kept for its later lookups, including those
 * after a preemption).  The walk, promotions, insertions and evictions are those of
 * eakv_tier_step with save(r) = `save`; the request is not registered again in the activity and
 * prompt-length windows of Eq. 10, which count first lookups, and it does not count as a request
 * in the statistics.  info_out->pressure is 0. */
int eakv_tier_step_again(eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks, int64_t n_tokens,
                         int64_t now_ms, int32_t save, uint8_t* hit_out, uint8_t* admit_out,
                         int32_t* slot_out, uint64_t* evicted_keys_out, int32_t* evicted_slots_out,
                         int64_t* n_evicted_inout, eakv_step_info* info_out);

/* Tier index export / import: carry a host tier across a restart of the process that owns the
 * context (no counterpart in the paper, whose replays start from a cold cache; Section 5.1).
 * eakv_tier_export writes the keys and slots of the resident units in recency order, least
 * recent first, into host arrays of `capacity` entries (either may be NULL) and the number of
 * residents into *n_out; E_CAPACITY if capacity is too small (nothing but *n_out is written).
 * eakv_tier_import fills the EMPTY host tier of a fresh context with such a list; together with
 * eakv_config.tier_memory pointing at the memory the old context used, the new context then
 * serves the same restores.  Slots handed out afterwards are the unused ones in ascending order,
 * as in a run that never evicted.  Not carried over: the GPU tier (the engine's blocks are gone
 * with the process), the counters, and the admission windows, which have a pair of calls of their
 * own below (without them they restart empty and capacity-conditioned admission may decide
 * differently until they refill).
 * The list names every unit the index holds, including those an open turn or request has admitted
 * but not written yet: for a restart, export when no turn or request is open (and after eakv_sync).
 * E_INVAL: tier not empty, a repeated key or slot, a slot outside the tier; nothing changes. */
int eakv_tier_export(const eakv_ctx* ctx, uint64_t* keys_host_out, int32_t* slots_host_out,
                     int64_t capacity, int64_t* n_out);
int eakv_tier_import(eakv_ctx* ctx, const uint64_t* keys_host, const int32_t* slots_host, int64_t n);

/* The admission windows (activity per agent, the last prompt lengths, eviction times: the inputs of
 * the pressure signal, Eq. 10) as an opaque list of int64 values, so that a restarted context decides
 * exactly as the old one would have.  Export: *n_out = number of values; values_host_out (may be
 * NULL) receives them if capacity suffices, else E_CAPACITY.  Import replaces the windows of a
 * context created with the same window settings; E_INVAL (nothing changes) on a malformed list. */
int eakv_admission_export(const eakv_ctx* ctx, int64_t* values_host_out, int64_t capacity, int64_t* n_out);
int eakv_admission_import(eakv_ctx* ctx, const int64_t* values_host, int64_t n);

/* The GPU tier's bookkeeping, which the paper leaves to the serving engine (Section 2):
 * an LRU of gpu_index_blocks keyed blocks referenced in order; a non-resident key takes
 * a block from a free stack (0, 1, 2, ... first; an evicted block is reused next).  With
 * need_tail a further unkeyed block is taken for the partial tail; give it back with
 * eakv_gpu_tier_release at the end of the turn.
 *   resident_out host uint8[n_blocks]; block_out host int32[n_blocks]; tail_block_out host
 * Errors: EAKV_E_CAPACITY when n_blocks + need_tail > gpu_index_blocks (nothing changes). */
int eakv_gpu_tier_step(eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks,
                       int32_t need_tail, uint8_t* resident_out, int32_t* block_out,
                       int32_t* tail_block_out);
int eakv_gpu_tier_release(eakv_ctx* ctx, int32_t block_id);

/* Several requests at once (Section 2: the engine runs up to a cap of requests at the same time
 * and suspends one if their KV no longer fits on the GPU; Appendix A: cap 16).  eakv_gpu_tier_acquire is
 * eakv_gpu_tier_step for a request that stays running: it references the keys in order in the same
 * way and then keeps every block of the prompt (and the tail block) pinned under request_id, out
 * of the recency order, so that no other request can take them.  A block already pinned by
 * another running request (a shared prefix) is shared.  EAKV_E_BUSY, nothing changed, when the
 * blocks nobody holds do not suffice: the caller waits, or suspends a running request with
 * eakv_gpu_tier_release_request and tries again.  EAKV_E_CAPACITY when the prompt could not be held
 * even with no other request running.  eakv_gpu_tier_release_request lets a finished
 * or suspended request's blocks go: those no other request holds re-enter the recency order at
 * the most-recent end in prompt order (tail first under EAKV_FREE_REVERSE) and keep their keys, so a
 * resumed request finds what has not been evicted meanwhile; the tail block is freed.  With one
 * request at a time acquire + release leaves the tier exactly as eakv_gpu_tier_step does.  While
 * any request holds blocks, eakv_gpu_tier_step and eakv_turn_begin return EAKV_E_INVAL.
 * Errors: EAKV_E_INVAL (request_id already holds blocks / holds none). */
int eakv_gpu_tier_acquire(eakv_ctx* ctx, int64_t request_id, const uint64_t* hashes_host, int64_t n_blocks,
                          int32_t need_tail, uint8_t* resident_out, int32_t* block_out,
                          int32_t* tail_block_out);
int eakv_gpu_tier_release_request(eakv_ctx* ctx, int64_t request_id);

/* Store (Section 2 host writes; Appendix D: a chunk is copied only if the tier lacks it, straight
 * out of the paged blocks that hold it): for every j with admit_mask[j] != 0 copy all 2L pieces of pool block
 * block_table[j] to tier slot host_slots[j].  admit_mask NULL = all admitted.
 *   block_table, host_slots host int32[n_blocks]; admit_mask host uint8[n_blocks] or NULL
 * Entries with admit 0 are ignored (their ids are not validated).  Asynchronous on
 * cuda_stream; with EAKV_LINK_STAGED the copy-engine part runs on a side stream that
 * cuda_stream waits for before the call's work counts as complete.
 * Errors: EAKV_E_RANGE, EAKV_E_INVAL (two admitted entries share a slot), EAKV_E_CUDA. */
int eakv_store(eakv_ctx* ctx, const int32_t* block_table, const uint8_t* admit_mask,
               const int32_t* host_slots, int64_t n_blocks, void* cuda_stream);

/* Load / restore (Section 3.1, the R * beta / B_H2D term of Eq. 3): copy all 2L pieces of
 * tier slot host_slots[j] into pool block block_table[j], for every j.
 * Errors: EAKV_E_RANGE, EAKV_E_INVAL (two entries share a destination block), EAKV_E_CUDA. */
int eakv_load(eakv_ctx* ctx, const int32_t* host_slots, const int32_t* block_table,
              int64_t n_blocks, void* cuda_stream);

/* One agent turn in two calls (the order of Section 4 and Appendix D: lookup when the request is
 * scheduled, restore before compute, store after compute).
 *
 * eakv_turn_begin: keys of the prompt's full blocks (eakv_hash_blocks on an internal lookup
 * stream, so it never waits behind transfers; blocks whose keys the caller already knows from
 * the previous turn are not hashed again), eakv_match, eakv_tier_step, eakv_gpu_tier_step, then
 * eakv_load of the host-covered blocks [G, H) on cuda_stream.  With chunk_blocks = R > 1 the
 * host tier sees one key per full chunk.  *view describes the turn; its arrays live in the
 * context and stay valid until the next eakv_turn_begin.
 *   tokens        device-accessible int32[n_tokens] (pinned host memory is fine), readable now
 *   known_keys    host uint64[n_known] keys of the first n_known blocks, or NULL / 0
 * The engine then produces the KV of every block with needs_fill[j] = 1 into gpu_block[j]
 * (ordered after cuda_stream's load) and calls
 * eakv_turn_end: eakv_store of the admitted blocks on cuda_stream (with eakv_config.write_behind:
 * on a stream of the context, behind what cuda_stream holds so far), and release of the partial
 * tail's temporary block.  One turn per context at a time.
 * Errors: those of the calls above; EAKV_E_INVAL when a turn is already open (begin) or none
 * is (end, abort).  eakv_turn_begin refuses what it can refuse (a prompt with more units than the
 * host tier, or more blocks than the GPU tier can hand out: EAKV_E_CAPACITY) before either tier
 * changes.  If a CUDA call fails after the bookkeeping (the restore in begin, the store in end),
 * no turn stays open and what the turn registered without producing it is taken back: the units
 * it admitted leave the host index and, in begin, the GPU blocks it newly keyed leave the GPU
 * index, so that no later lookup is answered from memory that was never written.  Promotions
 * and evictions the turn caused stand.
 * eakv_turn_abort closes an open turn whose KV the engine will not produce (a cancelled or
 * preempted request): admitted units and the blocks flagged needs_fill are taken back in the same
 * way, restored blocks stay, the tail block is released; nothing is stored.
 * A context created with control_plane_only runs the same two calls as pure bookkeeping (no
 * restore, no store) provided the caller passes all of the prompt's keys in known_keys.
 * eakv_turn_begin hashes on the context's own stream with the context's hash scratch: do not
 * run eakv_hash_blocks of the same context concurrently with it. */
typedef struct eakv_turn_view {
    int64_t n_blocks;             /* full blocks of the prompt                              */
    int64_t n_units;              /* tier units (= n_blocks / chunk_blocks)                 */
    int64_t gpu_prefix_blocks;    /* G                                                      */
    int64_t host_prefix_blocks;   /* H in blocks (host-covered units * chunk_blocks)        */
    int64_t restore_lo, restore_hi; /* blocks [lo, hi) restored from the host               */
    int64_t fresh_tokens;         /* n_tokens - max(G, H) * block_size                      */
    int64_t new_chunks;           /* u of the write rule                                    */
    int64_t n_fill, n_stored_blocks, n_evicted;
    int32_t pressure, save, tail_block, reserved;
    const uint64_t* keys;         /* [n_blocks]                                             */
    const int32_t*  gpu_block;    /* [n_blocks] pool block of every prompt block            */
    const uint8_t*  gpu_resident; /* [n_blocks] was resident when referenced                */
    const uint8_t*  needs_fill;   /* [n_blocks] the engine must compute this block's KV     */
    const uint8_t*  hit;          /* [n_units]                                              */
    const uint8_t*  admit;        /* [n_units]                                              */
    const int32_t*  slot;         /* [n_units] tier unit slot, -1 = declined                */
    const uint64_t* evicted_keys; /* [n_evicted]                                            */
    const int32_t*  evicted_slots;/* [n_evicted]                                            */
} eakv_turn_view;
int eakv_turn_begin(eakv_ctx* ctx, const int32_t* tokens, int64_t n_tokens,
                    const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                    void* cuda_stream, eakv_turn_view* view);
/* eakv_turn_begin with the restore in layer groups (eakv_load_layers): events[g] is recorded on
 * cuda_stream once group g of the restored blocks has landed -- also when the turn restores
 * nothing, so that a consumer may always wait on them.  A wrong n_events or a NULL event is
 * refused with EAKV_E_INVAL before anything changes.  (A bookkeeping-only context records nothing.) */
int eakv_turn_begin_layers(eakv_ctx* ctx, const int32_t* tokens, int64_t n_tokens,
                           const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                           int32_t layers_per_group, void* const* events, int32_t n_events,
                           void* cuda_stream, eakv_turn_view* view);
int eakv_turn_end(eakv_ctx* ctx, void* cuda_stream);
/* eakv_turn_end with the host write in layer groups (eakv_store_layers: group g is read only
 * after ready_events[g], which the engine recorded behind the work that completes those layers).
 * A wrong n_events is refused with EAKV_E_INVAL and the turn stays open. */
int eakv_turn_end_layers(eakv_ctx* ctx, int32_t layers_per_group, void* const* ready_events,
                         int32_t n_events, void* cuda_stream);
int eakv_turn_abort(eakv_ctx* ctx);

/* The same turn for an engine that runs several requests at once (Section 2: the engine's cap on
 * running requests; Appendix A: 16) and suspends one if their KV no longer fits on the GPU.  Any number of
 * requests may be open, each under a request_id of the caller's choosing.
 * eakv_request_begin: as eakv_turn_begin, but the prompt's GPU blocks are taken with
 * eakv_gpu_tier_acquire and stay pinned under request_id.  EAKV_E_BUSY, with neither tier
 * changed, when they do not fit beside the running requests: wait, or suspend a running request
 * (eakv_request_release) and try again (EAKV_E_CAPACITY: the prompt exceeds a tier on its own).  decided: -1 for the request's first lookup; 0 / 1 for a
 * later lookup of a resumed request, carrying the skip / store choice of its first one (Appendix D;
 * see eakv_tier_step_again).  *view's arrays stay valid until the request is released.
 * eakv_request_store: after the engine has produced the blocks flagged needs_fill, eakv_store of
 * the admitted blocks on cuda_stream (deferred under eakv_config.write_behind); once per begin.
 * Between a request's begin and its store the units it admitted are listed in the host tier (no
 * other request stores them again) but do not count toward another request's host prefix: their
 * slots hold nothing yet, so that request computes those blocks itself.  If another request's
 * lookup evicts such a unit before its store, the slot has a new owner and the store leaves that
 * unit out (view->n_stored_blocks counts what was admitted at the lookup; eakv_stats.blocks_stored
 * what was written); the bookkeeping is that of the reference model either way, which registers a
 * write at its lookup.  A release before the store takes back only the units the request still
 * owns.  After the store they are
 * restorable (a restore enqueued on another stream waits for that store).  The GPU side has
 * no such guard: a block that an open request was told to fill counts as resident for a later
 * request with the same prefix (the two share it), so an engine that runs both must let the
 * second one read that block only after the first one's fill (stream order or an event).
 * eakv_request_release: the request finished or is suspended: its blocks become evictable
 * (eakv_gpu_tier_release_request) and its tail block is freed.  Released before its store -- the
 * engine never produced the KV -- it is taken back like an aborted turn; a block it was told to fill
 * that another open request shares stays keyed for that request, which was told the block is
 * resident: the engine must then produce it on that request's behalf (or release that request too).
 * Errors: EAKV_E_INVAL for a request_id that is already open (begin) or not open (store, release),
 * for a second store, and while a single turn (eakv_turn_begin) is open; failures after the
 * bookkeeping are handled as in eakv_turn_begin / eakv_turn_end and close the request. */
int eakv_request_begin(eakv_ctx* ctx, int64_t request_id, const int32_t* tokens, int64_t n_tokens,
                       const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                       int32_t decided, void* cuda_stream, eakv_turn_view* view);
/* eakv_request_begin with the restore in layer groups, as eakv_turn_begin_layers. */
int eakv_request_begin_layers(eakv_ctx* ctx, int64_t request_id, const int32_t* tokens, int64_t n_tokens,
                              const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                              int32_t decided, int32_t layers_per_group, void* const* events, int32_t n_events,
                              void* cuda_stream, eakv_turn_view* view);
int eakv_request_store(eakv_ctx* ctx, int64_t request_id, void* cuda_stream);
/* eakv_request_store in layer groups, as eakv_turn_end_layers. */
int eakv_request_store_layers(eakv_ctx* ctx, int64_t request_id, int32_t layers_per_group,
                              void* const* ready_events, int32_t n_events, void* cuda_stream);
int eakv_request_release(eakv_ctx* ctx, int64_t request_id);

/* Layer-pipelined restore (Section 3.1, Eq. 2: the fixed restoration overhead tau_load is
 * what a consumer waits for before it can start; moving layers in order lets it start on
 * the first ones while the rest are in flight).  Same result as eakv_load, but the 2L
 * pieces of every block are moved in ascending groups of layers_per_group layers, and
 * events[g] is recorded on cuda_stream as soon as group g of all blocks has landed.
 *   events    host array of n_events cudaEvent_t handles (as void*), created by the caller;
 *             n_events must equal ceil(num_layers / layers_per_group)
 * A consumer stream that waits on events[g] may read layers g*layers_per_group .. of the
 * blocks in block_table.  Errors as eakv_load, plus EAKV_E_INVAL for a wrong n_events. */
int eakv_load_layers(eakv_ctx* ctx, const int32_t* host_slots, const int32_t* block_table,
                     int64_t n_blocks, int32_t layers_per_group, void* const* events,
                     int32_t n_events, void* cuda_stream);

/* Layer-pipelined host write (Section 3.1: write costs are part of what a response waits for
 * beyond its prefill; an engine that produces KV layer by layer can let the write of the first
 * layers run under the compute of the later ones).  Same result as eakv_store, but the 2L pieces
 * of every admitted block are moved in ascending groups of layers_per_group layers, and before
 * group g is read cuda_stream waits for ready_events[g].
 *   ready_events  host array of n_events cudaEvent_t handles (as void*) or NULL entries (no wait);
 *                 n_events must equal ceil(num_layers / layers_per_group).  The producer must
 *                 have recorded event g (cudaEventRecord already called, on its own stream,
 *                 behind the work that completes those layers of the blocks in block_table)
 *                 before this call: a wait on an event that was never recorded does not wait.
 * Errors as eakv_store, plus EAKV_E_INVAL for a wrong n_events. */
int eakv_store_layers(eakv_ctx* ctx, const int32_t* block_table, const uint8_t* admit_mask,
                      const int32_t* host_slots, int64_t n_blocks, int32_t layers_per_group,
                      void* const* ready_events, int32_t n_events, void* cuda_stream);

/* Reuse (stack) distances of a reference stream (Section 3.2, Eq. 4): dist[i] = number of
 * distinct other keys referenced strictly between reference i and the previous reference to
 * the same key, or -1 on a first reference.  Under a fully associative LRU tier of K chunks
 * that admits every miss, reference i hits iff 0 <= dist[i] < K.
 *   keys_dev device uint64[n_refs] (values below 2^61); dist_dev device int64[n_refs] (written)
 * Context-free.  Allocates its scratch (about (4 * ceil(log2 n) + 40) bytes per reference) with
 * cudaMalloc and frees it before returning; returns after the stream has finished the work.
 * n_refs < 2^31 - 16.  Errors: EAKV_E_INVAL, EAKV_E_CUDA (allocation or launch failure). */
int eakv_reuse_distances(const uint64_t* keys_dev, int64_t n_refs, int64_t* dist_dev,
                         void* cuda_stream);

/* Capacity curve from reuse distances (Appendix C "Prefix coverage from a reference stream"):
 * for every capacity K_c, hits = #{i : 0 <= dist[i] < K_c}; per request j (references
 * req_offsets[j] .. req_offsets[j+1]) the host coverage H_j is its leading run of hits,
 * restored += max(0, H_j - G_j) blocks and computed += n_j - max(G_j, H_j) * block_size tokens.
 *   dist_dev device int64[n_refs]; req_offsets_host int64[n_requests + 1] (0 .. n_refs);
 *   req_tokens_host, req_gpu_prefix_host int64[n_requests] (n_j and G_j in blocks);
 *   capacities_host int64[n_capacities], n_capacities <= 64;
 *   hits_out, restored_out, computed_out host int64[n_capacities];
 *   cover_out host int64[n_capacities][n_requests] (H_j per capacity) or NULL.
 * Context-free, allocates and frees its small scratch, returns after the work is done. */
int eakv_capacity_curve(const int64_t* dist_dev, int64_t n_refs, const int64_t* req_offsets_host,
                        const int64_t* req_tokens_host, const int64_t* req_gpu_prefix_host,
                        int64_t n_requests, int32_t block_size, const int64_t* capacities_host,
                        int32_t n_capacities, int64_t* hits_out, int64_t* restored_out,
                        int64_t* computed_out, int64_t* cover_out, void* cuda_stream);

/* Working-set sizes read off the reuse distances (Section 3.2, Section 5.4: where more host
 * capacity stops paying).  *full_out = largest finite distance + 1, the smallest tier (in tier
 * units) that hits every re-reference; *within_out = the smallest tier whose predicted computed
 * prefill (as eakv_capacity_curve computes it) is within `percent` per cent of the unbounded tier's.
 * Arguments as eakv_capacity_curve; context-free; returns after the work is done. */
int eakv_working_set_sizes(const int64_t* dist_dev, int64_t n_refs, const int64_t* req_offsets_host,
                           const int64_t* req_tokens_host, const int64_t* req_gpu_prefix_host,
                           int64_t n_requests, int32_t block_size, int32_t percent,
                           int64_t* full_out, int64_t* within_out, void* cuda_stream);

/* Declined-chunk audit (Appendix D, "Reuse distance of declined chunks"; Proposition 1): of the
 * references whose miss an admission policy declined, how many could be declined at no cost --
 * the chunk's next reference has reuse distance D >= capacity, or there is none.
 *   keys_dev      device uint64[n_refs], the tier's reference stream (values below 2^61)
 *   declined_dev  device uint8[n_refs], non-zero where the miss was declined
 *   capacity      K_H in tier units
 *   declined_out, meets_out, never_out  host: declined references, those meeting the condition,
 *                 those never referenced again (counted in meets_out too)
 *   next_dist_dev device int64[n_refs] or NULL: per reference, D of the next reference to its
 *                 chunk if it was declined (-1: never referenced again), -2 if it was not declined
 * Context-free; allocates its scratch (as eakv_reuse_distances, plus 12 bytes per reference) and
 * frees it before returning; returns after the stream has finished.  Errors as eakv_reuse_distances. */
int eakv_declined_audit(const uint64_t* keys_dev, const uint8_t* declined_dev, int64_t n_refs,
                        int64_t capacity, int64_t* declined_out, int64_t* meets_out, int64_t* never_out,
                        int64_t* next_dist_dev, void* cuda_stream);

/* Sizing arithmetic of Section 2 and Section 3.2 in integers (host only, no CUDA call):
 * beta_rank = 2 L d s max(1, ceil(H_kv / TP)) (Eq. 1); the working-set scale
 * C_reuse = (A - 1) * N_bar * beta_rank (Eq. 5) with N_bar = total_prompt_tokens / n_requests kept
 * as a fraction until the final floor; the pressure ratios gamma_G = A * N_bar / K_G with
 * K_G = gpu_blocks * block_size tokens and gamma_H = C_reuse / C_H with
 * C_H = host_blocks * block_size * beta_rank.  The two flags compare the fractions exactly
 * (gamma > 1); the doubles are for display.  A zero gpu_blocks / host_blocks leaves its ratio 0. */
typedef struct eakv_working_set_in {
    int32_t num_layers, kv_heads, head_dim, elem_bytes, tensor_parallel, block_size;
    int64_t active_pool;             /* A                                         */
    int64_t total_prompt_tokens;     /* sum of the prompt lengths of n_requests   */
    int64_t n_requests;
    int64_t gpu_blocks, host_blocks; /* K_G and K_H in blocks of block_size       */
} eakv_working_set_in;
typedef struct eakv_working_set_out {
    int64_t beta_rank_bytes;         /* Eq. 1                                     */
    int64_t working_set_bytes;       /* Eq. 5, floor                              */
    int64_t working_set_blocks;      /* floor(C_reuse / (block_size * beta_rank)) */
    double gamma_g, gamma_h;
    int32_t pool_exceeds_gpu;        /* gamma_G > 1                               */
    int32_t working_set_exceeds_host;/* gamma_H > 1                               */
} eakv_working_set_out;
int eakv_working_set(const eakv_working_set_in* in, eakv_working_set_out* out);

/* Offload benefit of Section 3.1, Eq. 2, in integers (host only, no CUDA call): restoring a prefix
 * of n tokens costs T_load(n) = n * beta_rank / B_H2D + tau_load, recomputing it T_rec(n) = n * t_pf;
 * OBR(n) = 1 - T_load(n) / T_rec(n).  Times in picoseconds (the paper's 0.86 us of restore per
 * token is 860,000).  obr_long_prefix is the limit 1 - beta_rank / (B_H2D * t_pf); break_even_tokens
 * the shortest prefix whose restore is not slower than its recomputation, -1 if there is none. */
typedef struct eakv_offload_in {
    int64_t prefix_tokens;           /* n                                           */
    int64_t beta_rank_bytes;         /* KV bytes per token and rank (Eq. 1)         */
    int64_t t_prefill_ps;            /* t_pf: prefill time per token, picoseconds   */
    int64_t h2d_bytes_per_s;         /* B_H2D                                       */
    int64_t tau_load_ps;             /* fixed cost of one restoration, picoseconds  */
} eakv_offload_in;
typedef struct eakv_offload_out {
    int64_t t_load_ps, t_rec_ps;
    int64_t break_even_tokens;
    double obr, obr_long_prefix;
    int32_t restore_is_faster;       /* T_load(n) < T_rec(n), compared exactly       */
    int32_t reserved;
} eakv_offload_out;
int eakv_offload_benefit(const eakv_offload_in* in, eakv_offload_out* out);

/* Block keys without a context and without any allocation.  (The paper has no counterpart;
 * this exists for callers that cannot request device memory: code living inside a serving
 * process whose engine has already claimed the GPU's memory, where an allocation may fail or
 * stall the device, and latency-critical sections that cannot afford an allocation's implicit
 * synchronisation.)  Same keys as eakv_hash_blocks for the same tokens, block_size, hash_base
 * (0 = library default) and parent_hash (pass the seed for a fresh prompt).
 *   tokens_dev device int32[n_tokens]; hashes_dev device uint64[n_tokens / block_size];
 *   n_blocks_out host or NULL; cuda_stream as elsewhere.
 * The scratch is a fixed array inside the library (about 545 KiB per GPU, held from the moment
 * the GPU loads the library's device code until the process exits) sized for at most
 * EAKV_STATIC_MAX_BLOCKS keys per call: a longer prompt gets EAKV_E_CAPACITY and nothing is
 * launched; hash it in pieces, passing the last key of one piece as parent_hash of the next.
 * The first call on each device looks up the array's device address (with that device
 * current).  Under the CUDA runtime's lazy loading that first call may also be what loads the
 * device code, array included, so make it once per device at start-up -- before the engine
 * claims the memory, outside any stream capture; a zero-length warm-up is not enough, pass at
 * least one block.  Concurrent first calls from several host threads are safe.
 * Every call on a device shares the array: calls whose GPU work can overlap race, so order
 * them (one stream, or events).  Calls no cudaMalloc/cudaFree or other allocating routine.
 * Errors: EAKV_E_INVAL (bad sizes/pointers, block_size > 4096), EAKV_E_CAPACITY, EAKV_E_CUDA.
 *
 * eakv_hash_blocks_static_status: the kernels behind the call above check every tile against the
 * sizes they were given and, instead of touching memory outside them, skip the tile and raise a
 * word in the same fixed array (the context-bound calls report this through eakv_sync).  This
 * call waits for cuda_stream, reads that word and returns EAKV_OK, or EAKV_E_RANGE after clearing
 * it: then keys of some call since the last query are missing.  Allocates nothing either. */
#define EAKV_STATIC_MAX_BLOCKS 65536
int eakv_hash_blocks_static(const int32_t* tokens_dev, int64_t n_tokens, int32_t block_size,
                            uint64_t hash_base, uint64_t parent_hash, uint64_t* hashes_dev,
                            int64_t* n_blocks_out, void* cuda_stream);
int eakv_hash_blocks_static_status(void* cuda_stream);

/* Block the host until everything the context enqueued (side streams included) is done. */
int eakv_sync(eakv_ctx* ctx);

/* Self-tests of the device-side checks (no counterpart in the paper).  Every kernel of the
 * library compares each entry / tile with the sizes of the buffers it was given and, instead of
 * touching memory outside them, skips it and raises an error word that the next eakv_sync
 * reports (EAKV_E_RANGE, or EAKV_E_TIMEOUT for a bounded wait that gave up) and clears.  The host
 * validates every id first, so in normal use these checks never trip; the two calls below make
 * them trip on purpose without any access out of bounds and without any unbounded wait.
 * eakv_selfcheck_limits: the kernels check against these NARROWER limits (pool blocks, tier
 * slots, keys per hash launch) until called again with zeros; values above the real sizes are
 * refused (EAKV_E_INVAL).  An entry between the narrowed and the real limit is then skipped on the
 * device: its bytes do not move, the rest of the call does (one exception: a store under
 * EAKV_LINK_STAGED gathers into a staging buffer that the copy engine moves as a whole, so the
 * slot of a skipped entry receives whatever that part of the staging buffer held).
 * eakv_selfcheck_wait_probe: enqueues a one-thread kernel that waits, with a short poll limit, on a
 * barrier nothing arrives at, gives up and raises the word: the next eakv_sync returns
 * EAKV_E_TIMEOUT and the context stays usable.
 * eakv_selfcheck_fail_next_transfer: a failure made on the host, for the paths that only a CUDA
 * error reaches otherwise: the next restore step of eakv_turn_begin / eakv_request_begin, or the
 * next store step of eakv_turn_end / eakv_request_store, returns `code` (a negative EAKV_E_*; 0
 * disarms) with nothing enqueued, once.  The call then behaves as after a real failure at that
 * point: what the turn registered is withdrawn.  Works on bookkeeping-only contexts too. */
int eakv_selfcheck_fail_next_transfer(eakv_ctx* ctx, int32_t code);
int eakv_selfcheck_limits(eakv_ctx* ctx, int64_t gpu_blocks, int64_t tier_slots, int64_t hash_blocks);
int eakv_selfcheck_wait_probe(eakv_ctx* ctx, void* cuda_stream);

int eakv_get_stats(const eakv_ctx* ctx, eakv_stats* out);
/* Base address of the tier (host pointer for TIER_PINNED_HOST, device pointer otherwise). */
void* eakv_tier_ptr(const eakv_ctx* ctx);
uint64_t eakv_hash_seed(const eakv_ctx* ctx);
uint64_t eakv_hash_base(const eakv_ctx* ctx);
const char* eakv_strerror(int code);
const char* eakv_last_cuda_error(const eakv_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* EAKV_H */
