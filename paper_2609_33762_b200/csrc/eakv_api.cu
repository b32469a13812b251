// C-ABI of libeakv: argument validation, host control plane, stream/event choreography.
// All data movement and hashing happens in the kernels of hash_kernels.cu /
// copy_kernels.cu (and, for the staged strategy, the copy engines); there is no CPU
// fallback: without a CUDA device eakv_create fails.
#include "../../include/eakv.h"

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <unordered_map>
#include <unordered_set>
#include <vector>

#include "control_plane.h"
#include "eakv_internal.h"

using namespace eakv;

namespace {

constexpr uint64_t P61 = (1ull << 61) - 1;
constexpr uint64_t kDefaultBase = 6364136223846793005ull % P61;
constexpr uint64_t kDefaultSeed = 0x9E3779B97F4A7C15ull % P61;
constexpr int kRingSlots = 8;

inline uint64_t mulmod_host(uint64_t a, uint64_t b) {
    return (uint64_t)(((unsigned __int128)a * b) % P61);
}

struct RingSlot {
    void* host = nullptr;     // pinned
    void* dev = nullptr;
    cudaEvent_t done = nullptr;   // recorded after the last consumer of the slot was enqueued
};

struct Staging {
    char* buf[2] = {nullptr, nullptr};
    cudaEvent_t ready[2] = {nullptr, nullptr};   // buffer filled
    cudaEvent_t freed[2] = {nullptr, nullptr};   // buffer drained
    cudaEvent_t start = nullptr;
    cudaStream_t side = nullptr;
    int next = 0;
};

}  // namespace

namespace {
constexpr int64_t kNoRequest = INT64_MIN;       // the single-turn calls are not bound to a request id

// what one open turn registered: its keys, both tiers' decisions, the per-block store plan
struct TurnState {
    std::vector<uint64_t> keys, unit_keys, evicted_keys;
    std::vector<int32_t> block, slot_u, slot_b, evicted_slots, host_slots;
    std::vector<uint8_t> resident, fill, hit, admit_u, admit_b;
    std::vector<uint8_t> owned_u;      // units this turn admitted and still has to write (see claim_units)
    int64_t request_id = kNoRequest;
    int32_t tail = -1;
    bool open = false, stored = false, claimed = false;
};
}  // namespace

// Which transfers of one direction may still be running, by tier slot.  Every transfer gets a
// sequence number; an event is recorded behind it in ring slot (number mod ring size) and the tier
// slots it touches remember the number.  When a ring slot is reused, the new event is recorded
// behind a wait for the old one, so whatever event a ring slot holds completes only after every
// earlier transfer that used that ring slot.  `done` trails the numbers known to be complete.
struct SlotOrder {
    static constexpr int kRing = 16;
    bool by_block = false;                 // index by pool block (ent[].x) instead of tier slot (ent[].y)
    cudaEvent_t ev[kRing] = {};
    cudaStream_t ev_stream[kRing] = {};
    uint64_t next = 1, done = 0;
    std::vector<uint64_t> slot_seq;        // by tier slot: the last transfer that touched it (0: none)

    // after a transfer over the slots ent[].y was enqueued on `stream`
    cudaError_t enqueued(const std::vector<int2>& ent, int64_t tier_slots, cudaStream_t stream) {
        if (slot_seq.empty()) slot_seq.assign((size_t)tier_slots, 0);
        // keep `done` moving also when nothing of the other direction asks for a long time
        for (int i = 0; i < 4 && done + 1 < next && cudaEventQuery(ev[(done + 1) % kRing]) == cudaSuccess; ++i) ++done;
        cudaGetLastError();                                // cudaErrorNotReady is not an error here
        const uint64_t seq = next++;
        const int idx = (int)(seq % kRing);
        cudaError_t e = cudaSuccess;
        if (!ev[idx]) e = cudaEventCreateWithFlags(&ev[idx], cudaEventDisableTiming);
        else if (ev_stream[idx] != stream) e = cudaStreamWaitEvent(stream, ev[idx], 0);
        if (e != cudaSuccess) return e;
        e = cudaEventRecord(ev[idx], stream);
        if (e != cudaSuccess) return e;
        ev_stream[idx] = stream;
        for (const int2& x : ent) slot_seq[by_block ? x.x : x.y] = seq;
        return cudaSuccess;
    }
    // before a transfer of the other direction over these slots is enqueued on `stream`: wait for
    // the transfers that touched them, unless complete or recorded on `stream` itself (in order)
    cudaError_t order_after(const std::vector<int2>& ent, cudaStream_t stream, bool forget) {
        if (slot_seq.empty()) return cudaSuccess;
        while (done + 1 < next && cudaEventQuery(ev[(done + 1) % kRing]) == cudaSuccess) ++done;
        cudaGetLastError();                                // cudaErrorNotReady is not an error here
        bool need[kRing] = {};
        bool any = false;
        for (const int2& x : ent) {
            uint64_t& q = slot_seq[by_block ? x.x : x.y];
            if (q > done) { need[q % kRing] = true; any = true; }
            if (forget) q = 0;
        }
        if (!any) return cudaSuccess;
        for (int idx = 0; idx < kRing; ++idx) {
            if (!need[idx] || ev_stream[idx] == stream) continue;
            const cudaError_t e = cudaStreamWaitEvent(stream, ev[idx], 0);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    }
    void destroy() {
        for (cudaEvent_t& e : ev)
            if (e) { cudaEventDestroy(e); e = nullptr; }
    }
};

struct eakv_ctx {
    eakv_config cfg;
    int device = 0;
    int sm_count = 0;
    int32_t pieces = 0;
    int64_t piece_bytes = 0, block_bytes = 0;
    uint64_t base = 0, seed = 0;

    void** d_kv_base = nullptr;
    char* pool_base = nullptr;     // kv_base[0]
    int64_t pool_pitch = 0;        // bytes between consecutive piece arrays when constant, else 0
    char* tier = nullptr;
    bool tier_owned = false;

    KeyedLru* host_tier = nullptr;
    KeyedLru* gpu_tier = nullptr;
    Admission* adm = nullptr;
    int64_t gpu_unkeyed = 0;
    struct HeldRequest { std::vector<int32_t> blocks; int32_t tail = -1; };
    std::unordered_map<int64_t, HeldRequest> held;     // running requests and the GPU blocks they pin
    eakv_stats stats;

    // hash
    uint64_t* d_pow = nullptr;
    std::vector<uint64_t> h_pow;   // B^0 .. B^b on the host
    uint64_t* d_partial = nullptr;
    int* d_counters = nullptr;
    int64_t hash_scratch_blocks = 0;
    int64_t max_prompts = 0;

    // argument rings
    RingSlot ring[kRingSlots];
    int ring_next = 0;
    size_t ring_bytes = 0;
    int64_t max_call_blocks = 0;

    // staged strategy
    Staging st_store, st_load;
    int64_t staging_blocks = 0;
    int64_t tier_slots = 0;        // block-sized slots in the tier = host_blocks * chunk_blocks
    int64_t chunk_tokens = 0;      // tokens per tier unit = block_size * chunk_blocks
    int64_t min_staged_run_bytes = 0;

    int* d_error_flag = nullptr;
    // limits the kernels check their entries / tiles against; narrower than the real sizes only
    // while eakv_selfcheck_limits is in force
    int64_t check_gpu_blocks = 0, check_tier_slots = 0, check_hash_blocks = 0;

    // duplicate-destination checks
    std::vector<uint32_t> slot_stamp, blk_stamp;
    uint32_t epoch = 0;
    std::vector<int2> scratch_entries;

    // two-call turn engine
    cudaStream_t lookup_stream = nullptr;
    // write-behind: the host write of a finished turn runs on wb_stream
    cudaStream_t wb_stream = nullptr;
    cudaEvent_t wb_fence = nullptr, wb_done = nullptr;
    bool wb_pending = false;
    std::vector<uint8_t> wb_blocks;     // by GPU block: a pending write still reads it
    std::vector<uint8_t> wb_slots;      // by tier slot: a pending write still fills it
    // Transfers in flight, by tier slot: a store into a slot that a restore on another stream may
    // still be reading waits for that restore, and a restore of a slot that a store on another
    // stream may still be writing waits for that store (Appendix D: the paper's tier exempts a
    // chunk with a copy in flight from eviction; here the bookkeeping may hand the slot on, and the
    // streams are ordered instead).
    SlotOrder restores, stores;
    // the same for pool blocks: a restore into (or an engine's fill of) a block that a store on
    // another stream may still be reading waits for that store
    SlotOrder block_reads;
    uint64_t* turn_keys = nullptr;            // pinned + mapped; the hash kernel writes it directly
    int64_t turn_keys_cap = 0;
    TurnState turn;                            // the one open turn of eakv_turn_begin / eakv_turn_end
    std::unordered_map<int64_t, TurnState> requests;   // open turns of running requests (eakv_request_*)
    // units an open request admitted and has not written yet -> that request.  An eviction takes a
    // unit out of here: its slot belongs to someone else from then on and is never written by the
    // request that lost it.  While listed here a unit is in the host index (nobody stores it twice)
    // but no other request can restore it.
    std::unordered_map<uint64_t, int64_t> unstored_units;
    int fail_next_transfer = 0;        // self-test: the next restore / store step returns this code instead

    std::string cuda_err;
};

namespace {

int cuda_fail(eakv_ctx* c, cudaError_t e, const char* what) {
    if (c) {
        c->cuda_err = std::string(what) + ": " + cudaGetErrorString(e);
    }
    return EAKV_E_CUDA;
}

#define CU(call)                                                    \
    do {                                                            \
        cudaError_t _e = (call);                                    \
        if (_e != cudaSuccess) return cuda_fail(ctx, _e, #call);    \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (dev >= 0 && cudaGetDevice(&prev) == cudaSuccess && prev != dev) {
            switched = cudaSetDevice(dev) == cudaSuccess;
        }
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

// Take the next ring slot; blocks only if its previous use (kRingSlots calls ago) is still
// pending on the GPU.
int ring_acquire(eakv_ctx* ctx, RingSlot** out) {
    RingSlot* s = &ctx->ring[ctx->ring_next];
    ctx->ring_next = (ctx->ring_next + 1) % kRingSlots;
    CU(cudaEventSynchronize(s->done));
    *out = s;
    return EAKV_OK;
}

void free_all(eakv_ctx* c) {
    if (!c) return;
    for (auto& s : c->ring) {
        if (s.host) cudaFreeHost(s.host);
        if (s.dev) cudaFree(s.dev);
        if (s.done) cudaEventDestroy(s.done);
    }
    for (Staging* st : {&c->st_store, &c->st_load}) {
        for (int i = 0; i < 2; ++i) {
            if (st->buf[i]) cudaFree(st->buf[i]);
            if (st->ready[i]) cudaEventDestroy(st->ready[i]);
            if (st->freed[i]) cudaEventDestroy(st->freed[i]);
        }
        if (st->start) cudaEventDestroy(st->start);
        if (st->side) cudaStreamDestroy(st->side);
    }
    if (c->d_kv_base) cudaFree(c->d_kv_base);
    if (c->d_pow) cudaFree(c->d_pow);
    if (c->d_partial) cudaFree(c->d_partial);
    if (c->d_counters) cudaFree(c->d_counters);
    if (c->d_error_flag) cudaFree(c->d_error_flag);
    if (c->turn_keys) cudaFreeHost(c->turn_keys);
    if (c->lookup_stream) cudaStreamDestroy(c->lookup_stream);
    if (c->wb_stream) cudaStreamDestroy(c->wb_stream);
    if (c->wb_fence) cudaEventDestroy(c->wb_fence);
    if (c->wb_done) cudaEventDestroy(c->wb_done);
    c->restores.destroy();
    c->stores.destroy();
    c->block_reads.destroy();
    if (c->tier && c->tier_owned) {
        if (c->cfg.tier_location == EAKV_TIER_DEVICE) cudaFree(c->tier);
        else cudaFreeHost(c->tier);
    }
    delete c->host_tier;
    delete c->gpu_tier;
    delete c->adm;
    delete c;
}

// grid of a kernel that touches the mapped host tier: per direction if configured
// A few SMs saturate the host link and the rest stay with the engine.  Measured with restores
// and writes running at once (zero-copy, 6 GiB each way, GB/s of both directions together):
// vector kernel both ways, one grid size: 16 CTAs 49.5, 32: 63.7, 64: 73-74, 128: 72.6, 296: 73.2;
// restores through the bulk-copy ring (load CTAs / store CTAs): 32/64 65.0, 48/64 70.5, 64/48 73.7,
// 64/64 78.1, 80/80 77.1, 96/64 78.8, 64/96 70.5, 64/128 63.0, 148/32 59.9 -- more writers starve
// the read requests, which share the upstream direction with the posted writes.  One direction
// alone is flat from 32 CTAs up (52 GB/s with either kernel).
int host_ctas(const eakv_ctx* ctx, bool to_tier) {
    const int dir = to_tier ? ctx->cfg.host_store_ctas : ctx->cfg.host_load_ctas;
    if (dir > 0) return dir;
    if (ctx->cfg.copy_ctas > 0) return ctx->cfg.copy_ctas;
    const bool bulk_load = !to_tier && ctx->cfg.host_copy_path != EAKV_HOST_COPY_VECTOR;
    return bulk_load ? 96 : 64;
}

// grid of the vector kernel: the configured one, else sized here
int vector_ctas(const eakv_ctx* ctx, bool touches_host) {
    if (ctx->cfg.copy_ctas > 0) return ctx->cfg.copy_ctas;
    (void)touches_host;
    return ctx->sm_count * copy_vector_ctas_per_sm();
}

// d_entries == NULL: the n (<= kCopyInlineEntries) entries at h_inline ride in the parameters
// [q_first, q_first + q_count): the piece arrays moved (all 2L, or one layer group)
int launch_copy(eakv_ctx* ctx, const int2* d_entries, const int2* h_inline, int64_t n,
                char* tier_base, bool to_tier, bool touches_host, bool packed, cudaStream_t stream,
                int q_first, int q_count, int64_t packed_capacity) {
    CopyLaunch L;
    L.entries = d_entries;
    if (!d_entries) std::memcpy(L.inline_entries, h_inline, (size_t)n * sizeof(int2));
    L.n_entries = n;
    L.kv_base = ctx->d_kv_base;
    L.tier_base = tier_base;
    L.pieces = q_count;
    L.q_first = q_first;
    L.slot_pieces = packed ? q_count : ctx->pieces;
    L.slot_q_first = packed ? 0 : q_first;
    L.piece_bytes = ctx->piece_bytes;
    L.slot_from_index = packed ? 1 : 0;
    L.gpu_blocks = ctx->check_gpu_blocks;
    L.tier_slots = packed ? packed_capacity : ctx->check_tier_slots;
    L.error_flag = ctx->d_error_flag;
    L.subs_per_piece = (int32_t)((ctx->piece_bytes + kCopySubBytes - 1) / kCopySubBytes);
    L.group_pieces = 1;          // the bulk launcher raises it for small pieces
    L.pad0 = 0;
    cudaError_t e;
    // a mapped host tier gets a small grid (a few SMs saturate the link) of the vector kernel or,
    // if configured, the bulk-copy ring; device-resident buffers get the configured copy path
    if (touches_host) {
        const bool bulk = ctx->cfg.host_copy_path == EAKV_HOST_COPY_BULK_BOTH ||
                          (ctx->cfg.host_copy_path == EAKV_HOST_COPY_BULK_LOAD && !to_tier);
        if (bulk) e = launch_copy_bulk(L, to_tier, host_ctas(ctx, to_tier), ctx->sm_count, stream);
        else      e = launch_copy_vector(L, to_tier, host_ctas(ctx, to_tier), stream);
    } else if (ctx->cfg.copy_path == EAKV_COPY_BULK) {
        e = launch_copy_bulk(L, to_tier, ctx->cfg.copy_ctas > 0 ? ctx->cfg.copy_ctas : 0, ctx->sm_count, stream);
    } else {
        e = launch_copy_vector(L, to_tier, vector_ctas(ctx, false), stream);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "copy kernel launch");
    ctx->stats.kernel_launches += 1;
    return EAKV_OK;
}

// Upload n entries through a ring slot.  *dev_out is valid for work enqueued on `stream`
// (and on streams ordered after it) until ring_release records the slot's event.
int ring_upload(eakv_ctx* ctx, const int2* entries, int64_t n, cudaStream_t stream,
                RingSlot** slot_out, const int2** dev_out) {
    RingSlot* s = nullptr;
    int rc = ring_acquire(ctx, &s);
    if (rc != EAKV_OK) return rc;
    std::memcpy(s->host, entries, (size_t)n * sizeof(int2));
    CU(launch_fetch_args(s->dev, s->host, (size_t)n * sizeof(int2), stream));
    ctx->stats.kernel_launches += 1;
    *slot_out = s;
    *dev_out = static_cast<const int2*>(s->dev);
    return EAKV_OK;
}

int ring_release(eakv_ctx* ctx, RingSlot* s, cudaStream_t stream) {
    CU(cudaEventRecord(s->done, stream));
    return EAKV_OK;
}

int next_epoch(eakv_ctx* ctx) {
    if (++ctx->epoch == 0) {   // wrapped: clear the stamps
        std::fill(ctx->slot_stamp.begin(), ctx->slot_stamp.end(), 0u);
        std::fill(ctx->blk_stamp.begin(), ctx->blk_stamp.end(), 0u);
        ctx->epoch = 1;
    }
    return EAKV_OK;
}

// contiguous runs of host slots inside a chunk: [i0, i1) with slots e[i0].y, e[i0].y+1, ...
template <class F>
int for_slot_runs(const int2* e, int64_t n, F f) {
    int64_t i0 = 0;
    while (i0 < n) {
        int64_t i1 = i0 + 1;
        while (i1 < n && e[i1].y == e[i1 - 1].y + 1) ++i1;
        int rc = f(i0, i1);
        if (rc != EAKV_OK) return rc;
        i0 = i1;
    }
    return EAKV_OK;
}


// Move the m compacted entries {pool block, tier slot} between pool and tier.
//   direct : the copy kernel addresses the tier itself (HBM tier, or mapped host tier)
//   staged : HBM staging buffers + copy engine on the side stream, double-buffered
// Under EAKV_LINK_STAGED a call whose slots are so scattered that the copy engine would get
// mostly single-block copies goes direct instead (per-copy overhead outweighs the DMA's edge).
// Order `stream` after a pending write-behind store (no-op when none is pending, when it has
// completed, or for the write-behind stream itself).
int wait_write_behind(eakv_ctx* ctx, cudaStream_t stream) {
    if (!ctx->wb_pending || stream == ctx->wb_stream) return EAKV_OK;
    if (cudaEventQuery(ctx->wb_done) == cudaSuccess) {
        ctx->wb_pending = false;
        std::fill(ctx->wb_blocks.begin(), ctx->wb_blocks.end(), (uint8_t)0);
        std::fill(ctx->wb_slots.begin(), ctx->wb_slots.end(), (uint8_t)0);
        return EAKV_OK;
    }
    cudaGetLastError();            // cudaErrorNotReady is not an error here
    CU(cudaStreamWaitEvent(stream, ctx->wb_done, 0));
    return EAKV_OK;
}

int move_blocks(eakv_ctx* ctx, const std::vector<int2>& ent, bool to_tier, cudaStream_t stream,
                int q_first, int q_count) {
    const int64_t m = (int64_t)ent.size();
    const bool whole = q_count == ctx->pieces;
    const int64_t range_bytes = (int64_t)q_count * ctx->piece_bytes;      // per block
    // a staging buffer holds more blocks when only a layer group of each is moved
    const int64_t stage_cap = whole ? ctx->staging_blocks
        : std::min<int64_t>(ctx->max_call_blocks, ctx->staging_blocks * ctx->block_bytes / range_bytes);
    const bool host_tier = ctx->cfg.tier_location == EAKV_TIER_PINNED_HOST;
    if (ctx->cfg.link_strategy == EAKV_LINK_COPY_ENGINE) {
        // one strided transfer per block: q_count rows of one piece, pool pitch against slot pitch
        for (int64_t i = 0; i < m; ++i) {
            char* pool_p = ctx->pool_base + (int64_t)q_first * ctx->pool_pitch + (int64_t)ent[i].x * ctx->piece_bytes;
            char* tier_p = ctx->tier + (int64_t)ent[i].y * ctx->block_bytes + (int64_t)q_first * ctx->piece_bytes;
            CU(cudaMemcpy2DAsync(to_tier ? tier_p : pool_p, to_tier ? (size_t)ctx->piece_bytes : (size_t)ctx->pool_pitch,
                                 to_tier ? pool_p : tier_p, to_tier ? (size_t)ctx->pool_pitch : (size_t)ctx->piece_bytes,
                                 (size_t)ctx->piece_bytes, (size_t)q_count, cudaMemcpyDefault, stream));
            ctx->stats.memcpy_calls += 1;
        }
        return EAKV_OK;
    }
    bool direct = ctx->cfg.link_strategy == EAKV_LINK_ZERO_COPY;
    if (!direct) {
        int64_t runs = 0;
        for_slot_runs(ent.data(), m, [&](int64_t, int64_t) { ++runs; return EAKV_OK; });
        const int64_t avg_run_bytes = m * range_bytes / runs;
        direct = avg_run_bytes < ctx->min_staged_run_bytes;
    }
    Staging& S = to_tier ? ctx->st_store : ctx->st_load;
    if (!direct && !to_tier) {
        // the side stream may read the tier only after what precedes this call on `stream`
        CU(cudaEventRecord(S.start, stream));
        CU(cudaStreamWaitEvent(S.side, S.start, 0));
    }
    for (int64_t base = 0; base < m; base += ctx->max_call_blocks) {
        const int64_t n = std::min(ctx->max_call_blocks, m - base);
        const int2* h = ent.data() + base;
        // small calls carry their entries in the kernel parameters: no upload, no ring slot
        const bool inline_args = n <= kCopyInlineEntries;
        RingSlot* rs = nullptr;
        const int2* d = nullptr;
        int rc = EAKV_OK;
        if (!inline_args) {
            rc = ring_upload(ctx, h, n, stream, &rs, &d);
            if (rc != EAKV_OK) return rc;
        }
        if (direct) {
            rc = launch_copy(ctx, d, h, n, ctx->tier, to_tier, host_tier, false, stream,
                             q_first, q_count, 0);
            if (rc != EAKV_OK) return rc;
        } else {
            for (int64_t i = 0; i < n; i += stage_cap) {
                const int64_t cur = std::min(stage_cap, n - i);
                const int sb = S.next;
                S.next ^= 1;
                const int2* e = h + i;
                auto dma = [&](int64_t a, int64_t z) {
                    char* tier_p = ctx->tier + (int64_t)e[a].y * ctx->block_bytes +
                                   (int64_t)q_first * ctx->piece_bytes;
                    char* stage_p = S.buf[sb] + a * range_bytes;
                    if (whole) {
                        CU(cudaMemcpyAsync(to_tier ? tier_p : stage_p, to_tier ? stage_p : tier_p,
                                           (size_t)(z - a) * ctx->block_bytes, cudaMemcpyDefault, S.side));
                    } else {   // one strip per slot: rows of range_bytes, slot pitch on the tier side
                        CU(cudaMemcpy2DAsync(to_tier ? tier_p : stage_p,
                                             to_tier ? (size_t)ctx->block_bytes : (size_t)range_bytes,
                                             to_tier ? stage_p : tier_p,
                                             to_tier ? (size_t)range_bytes : (size_t)ctx->block_bytes,
                                             (size_t)range_bytes, (size_t)(z - a), cudaMemcpyDefault, S.side));
                    }
                    ctx->stats.memcpy_calls += 1;
                    return EAKV_OK;
                };
                if (to_tier) {
                    CU(cudaStreamWaitEvent(stream, S.freed[sb], 0));
                    rc = launch_copy(ctx, d ? d + i : nullptr, e, cur, S.buf[sb], true, false, true, stream,
                                     q_first, q_count, stage_cap);
                    if (rc != EAKV_OK) return rc;
                    CU(cudaEventRecord(S.ready[sb], stream));
                    CU(cudaStreamWaitEvent(S.side, S.ready[sb], 0));
                    rc = for_slot_runs(e, cur, dma);
                    if (rc != EAKV_OK) return rc;
                    CU(cudaEventRecord(S.freed[sb], S.side));
                } else {
                    CU(cudaStreamWaitEvent(S.side, S.freed[sb], 0));
                    rc = for_slot_runs(e, cur, dma);
                    if (rc != EAKV_OK) return rc;
                    CU(cudaEventRecord(S.ready[sb], S.side));
                    CU(cudaStreamWaitEvent(stream, S.ready[sb], 0));
                    rc = launch_copy(ctx, d ? d + i : nullptr, e, cur, S.buf[sb], false, false, true, stream,
                                     q_first, q_count, stage_cap);
                    if (rc != EAKV_OK) return rc;
                    CU(cudaEventRecord(S.freed[sb], stream));
                }
            }
            if (to_tier) {
                // the call's work is complete, in stream order, once both buffers are drained
                CU(cudaStreamWaitEvent(stream, S.freed[0], 0));
                CU(cudaStreamWaitEvent(stream, S.freed[1], 0));
            }
        }
        if (rs) {
            rc = ring_release(ctx, rs, stream);
            if (rc != EAKV_OK) return rc;
        }
    }
    return EAKV_OK;
}

}  // namespace

extern "C" {

int eakv_config_init(eakv_config* cfg) {
    if (!cfg) return EAKV_E_INVAL;
    std::memset(cfg, 0, sizeof(*cfg));
    cfg->elem_bytes = 2;
    cfg->policy = EAKV_POLICY_WRITE_ALL;
    cfg->kappa_blocks = 8;
    cfg->theta_percent = 95;
    cfg->len_window = 256;
    cfg->window_ms = 60000;
    cfg->telemetry = 1;
    cfg->link_strategy = EAKV_LINK_STAGED;
    cfg->tier_location = EAKV_TIER_PINNED_HOST;
    cfg->copy_path = EAKV_COPY_BULK;
    cfg->host_copy_path = EAKV_HOST_COPY_BULK_LOAD;
    return EAKV_OK;
}

int eakv_create(const eakv_config* cfg, eakv_ctx** out) {
    if (!cfg || !out) return EAKV_E_INVAL;
    *out = nullptr;
    if (cfg->num_layers <= 0 || cfg->kv_heads <= 0 || cfg->head_dim <= 0 || cfg->block_size <= 0 ||
        cfg->elem_bytes <= 0 || cfg->gpu_blocks <= 0 || cfg->host_blocks <= 0 ||
        (!cfg->kv_base && !cfg->control_plane_only))
        return EAKV_E_INVAL;
    if (cfg->block_size > kHashMaxBlockSize) return EAKV_E_INVAL;
    const int64_t chunk_blocks = cfg->chunk_blocks > 0 ? cfg->chunk_blocks : 1;
    if (cfg->gpu_blocks > INT32_MAX || cfg->host_blocks > INT32_MAX / chunk_blocks) return EAKV_E_INVAL;
    if (cfg->policy < 0 || cfg->policy > 2 || cfg->link_strategy < 0 || cfg->link_strategy > 2 ||
        cfg->tier_location < 0 || cfg->tier_location > 1 || cfg->copy_path < 0 || cfg->copy_path > 1 ||
        cfg->gpu_free_order < 0 || cfg->gpu_free_order > 1)
        return EAKV_E_INVAL;
    if (cfg->gpu_index_blocks < 0 || cfg->gpu_index_blocks > cfg->gpu_blocks) return EAKV_E_INVAL;
    if (cfg->telemetry_period_ms < 0 || cfg->telemetry_max_age_ms < 0) return EAKV_E_INVAL;
    if (cfg->host_copy_path < 0 || cfg->host_copy_path > 2 || cfg->host_load_ctas < 0 || cfg->host_store_ctas < 0)
        return EAKV_E_INVAL;
    const int64_t piece = (int64_t)cfg->block_size * cfg->kv_heads * cfg->head_dim * cfg->elem_bytes;
    if (piece % 16 != 0) return EAKV_E_INVAL;
    const int pieces = 2 * cfg->num_layers;
    for (int q = 0; q < pieces && !cfg->control_plane_only; ++q) {
        if (!cfg->kv_base[q] || ((uintptr_t)cfg->kv_base[q] & 15)) return EAKV_E_INVAL;
    }
    if (cfg->tier_memory && ((uintptr_t)cfg->tier_memory & 15)) return EAKV_E_INVAL;

    int ndev = 0;
    if (!cfg->control_plane_only && (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0))
        return EAKV_E_CUDA;

    eakv_ctx* ctx = new (std::nothrow) eakv_ctx();
    if (!ctx) return EAKV_E_NOMEM;
    ctx->cfg = *cfg;
    ctx->cfg.kv_base = nullptr;
    // a tier in HBM is copied directly; staging only makes sense across the host link
    if (cfg->tier_location == EAKV_TIER_DEVICE && cfg->link_strategy == EAKV_LINK_STAGED)
        ctx->cfg.link_strategy = EAKV_LINK_ZERO_COPY;
    if (!cfg->control_plane_only) {
        ctx->pool_base = static_cast<char*>(cfg->kv_base[0]);
        int64_t pitch = pieces > 1 ? static_cast<char*>(cfg->kv_base[1]) - static_cast<char*>(cfg->kv_base[0]) : piece * cfg->gpu_blocks;
        for (int q = 1; q < pieces && pitch > 0; ++q)
            if (static_cast<char*>(cfg->kv_base[q]) - static_cast<char*>(cfg->kv_base[q - 1]) != pitch) pitch = 0;
        if (pitch < piece * cfg->gpu_blocks) pitch = 0;
        ctx->pool_pitch = pitch;
    }
    if (cfg->link_strategy == EAKV_LINK_COPY_ENGINE && (cfg->control_plane_only || ctx->pool_pitch == 0)) {
        delete ctx;
        return EAKV_E_INVAL;
    }
    if (cfg->link_strategy == EAKV_LINK_COPY_ENGINE) {
        // a strided copy-engine transfer takes no pitch above the device's limit (cudaDevAttrMaxPitch)
        int dev = 0, max_pitch = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&max_pitch, cudaDevAttrMaxPitch, dev) != cudaSuccess) {
            cudaGetLastError();
            delete ctx;
            return EAKV_E_CUDA;
        }
        if (ctx->pool_pitch > (int64_t)max_pitch || piece * pieces > (int64_t)max_pitch) {
            delete ctx;
            return EAKV_E_INVAL;
        }
    }
    std::memset(&ctx->stats, 0, sizeof(ctx->stats));
    ctx->pieces = pieces;
    ctx->piece_bytes = piece;
    ctx->block_bytes = piece * pieces;
    ctx->base = cfg->hash_base ? cfg->hash_base % P61 : kDefaultBase;
    ctx->seed = cfg->hash_seed ? cfg->hash_seed % P61 : kDefaultSeed;
    ctx->max_call_blocks = cfg->max_call_blocks > 0 ? cfg->max_call_blocks : 16384;
    ctx->hash_scratch_blocks = cfg->hash_scratch_blocks > 0 ? cfg->hash_scratch_blocks : (1 << 20);
    ctx->max_prompts = ctx->max_call_blocks;
    ctx->tier_slots = cfg->host_blocks * chunk_blocks;
    ctx->check_gpu_blocks = cfg->gpu_blocks;
    ctx->check_tier_slots = ctx->tier_slots;
    ctx->chunk_tokens = (int64_t)cfg->block_size * chunk_blocks;
    ctx->min_staged_run_bytes = cfg->min_staged_run_bytes >= 0 ? cfg->min_staged_run_bytes : 0;
    if (cfg->min_staged_run_bytes == 0) ctx->min_staged_run_bytes = 3ll << 20;

#define CUC(call)                                             \
    do {                                                      \
        cudaError_t _e = (call);                              \
        if (_e != cudaSuccess) {                              \
            int rc = (_e == cudaErrorMemoryAllocation) ? EAKV_E_NOMEM : EAKV_E_CUDA; \
            std::fprintf(stderr, "eakv_create: %s: %s\n", #call, cudaGetErrorString(_e)); \
            cudaGetLastError();                               \
            free_all(ctx);                                    \
            return rc;                                        \
        }                                                     \
    } while (0)

    if (!cfg->control_plane_only) {
        // the pool and an adopted tier are read and written by kernels: refuse addresses they cannot reach
        bool reachable = !cfg->tier_memory || device_readable(cfg->tier_memory);
        for (int q = 0; q < pieces && reachable; ++q) reachable = device_readable(cfg->kv_base[q]);
        if (!reachable) {
            free_all(ctx);
            return EAKV_E_INVAL;
        }
        CUC(cudaGetDevice(&ctx->device));
        CUC(cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device));
        CUC(hash_kernels_init());
        CUC(copy_kernels_init());
    }

    ctx->block_reads.by_block = true;
    try {
        ctx->host_tier = new KeyedLru(cfg->host_blocks);
        ctx->gpu_tier = new KeyedLru(cfg->gpu_index_blocks ? cfg->gpu_index_blocks : cfg->gpu_blocks);
        ctx->adm = new Admission(cfg->policy, cfg->kappa_blocks, cfg->theta_percent, cfg->window_ms,
                                 cfg->len_window > 0 ? cfg->len_window : 256, cfg->telemetry,
                                 cfg->host_blocks, cfg->block_size * (int32_t)chunk_blocks,
                                 cfg->telemetry_period_ms, cfg->telemetry_max_age_ms);
        ctx->slot_stamp.assign((size_t)ctx->tier_slots, 0);
        ctx->blk_stamp.assign((size_t)cfg->gpu_blocks, 0);
    } catch (const std::bad_alloc&) {
        free_all(ctx);
        return EAKV_E_NOMEM;
    }

    if (cfg->control_plane_only) {   // bookkeeping only: nothing below is needed
        ctx->device = -1;
        *out = ctx;
        return EAKV_OK;
    }

    // piece-array base pointers
    CUC(cudaMalloc(&ctx->d_kv_base, sizeof(void*) * pieces));
    CUC(cudaMemcpy(ctx->d_kv_base, cfg->kv_base, sizeof(void*) * pieces, cudaMemcpyHostToDevice));

    // tier memory
    const size_t tier_bytes = (size_t)ctx->tier_slots * (size_t)ctx->block_bytes;
    if (cfg->tier_memory) {
        ctx->tier = static_cast<char*>(cfg->tier_memory);
    } else if (cfg->tier_location == EAKV_TIER_DEVICE) {
        CUC(cudaMalloc(&ctx->tier, tier_bytes));
        ctx->tier_owned = true;
    } else {
        CUC(cudaHostAlloc(&ctx->tier, tier_bytes, cudaHostAllocMapped | cudaHostAllocPortable));
        ctx->tier_owned = true;
    }

    // hash: power table B^0..B^b, partial scratch, ticket counters
    {
        std::vector<uint64_t> pw((size_t)cfg->block_size + 1);
        pw[0] = 1;
        for (int e = 1; e <= cfg->block_size; ++e) pw[e] = mulmod_host(pw[e - 1], ctx->base);
        ctx->h_pow = pw;
        CUC(cudaMalloc(&ctx->d_pow, pw.size() * 8));
        CUC(cudaMemcpy(ctx->d_pow, pw.data(), pw.size() * 8, cudaMemcpyHostToDevice));
        CUC(cudaMalloc(&ctx->d_partial, (size_t)ctx->hash_scratch_blocks * 8));
        CUC(cudaMalloc(&ctx->d_counters, (size_t)ctx->max_prompts * sizeof(int)));
        CUC(cudaMemset(ctx->d_counters, 0, (size_t)ctx->max_prompts * sizeof(int)));
        CUC(cudaMalloc(&ctx->d_error_flag, sizeof(int)));
        CUC(cudaMemset(ctx->d_error_flag, 0, sizeof(int)));
    }

    // argument rings: room for max_call_blocks copy entries, or the batched-hash descriptors
    ctx->ring_bytes = std::max<size_t>((size_t)ctx->max_call_blocks * sizeof(HashPrompt) +
                                           (size_t)ctx->max_call_blocks * sizeof(HashTile),
                                       (size_t)1 << 16);
    for (auto& s : ctx->ring) {
        CUC(cudaHostAlloc(&s.host, ctx->ring_bytes, cudaHostAllocMapped | cudaHostAllocPortable));
        CUC(cudaMalloc(&s.dev, ctx->ring_bytes));
        CUC(cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming));
    }

    // staged strategy
    if (ctx->cfg.link_strategy == EAKV_LINK_STAGED) {
        // 256 MiB per buffer: with both directions busy the step moved 95.5 GB/s at 16 MiB, 97.4-98.6
        // at 32-128 MiB, 99.5 at 256 MiB and 99.9 at 512 MiB of a 100 GB/s two-way pinned rate
        int64_t sbytes = cfg->staging_bytes > 0 ? cfg->staging_bytes : (256ll << 20);
        ctx->staging_blocks = std::max<int64_t>(1, sbytes / ctx->block_bytes);
        ctx->staging_blocks = std::min(ctx->staging_blocks, ctx->max_call_blocks);
        // no call moves more blocks than the smaller of the pool and the tier holds
        ctx->staging_blocks = std::min(ctx->staging_blocks, std::min<int64_t>(ctx->tier_slots, cfg->gpu_blocks));
        for (Staging* st : {&ctx->st_store, &ctx->st_load}) {
            for (int i = 0; i < 2; ++i) {
                CUC(cudaMalloc(&st->buf[i], (size_t)ctx->staging_blocks * ctx->block_bytes));
                CUC(cudaEventCreateWithFlags(&st->ready[i], cudaEventDisableTiming));
                CUC(cudaEventCreateWithFlags(&st->freed[i], cudaEventDisableTiming));
            }
            CUC(cudaEventCreateWithFlags(&st->start, cudaEventDisableTiming));
            CUC(cudaStreamCreateWithFlags(&st->side, cudaStreamNonBlocking));
        }
    }
    CUC(cudaDeviceSynchronize());
#undef CUC
    *out = ctx;
    return EAKV_OK;
}

int eakv_sync(eakv_ctx* ctx) {
    if (!ctx) return EAKV_E_INVAL;
    if (ctx->device < 0) return EAKV_OK;
    DeviceGuard g(ctx->device);
    CU(cudaDeviceSynchronize());
    int flag = 0;
    CU(cudaMemcpy(&flag, ctx->d_error_flag, sizeof(int), cudaMemcpyDeviceToHost));
    if (flag != 0) {   // a device-side self-check tripped since the last sync
        CU(cudaMemset(ctx->d_error_flag, 0, sizeof(int)));
        CU(cudaMemset(ctx->d_counters, 0, (size_t)ctx->max_prompts * sizeof(int)));
        ctx->cuda_err = flag == kErrBulkTimeout ? "bulk-copy wait gave up"
                      : flag == kErrCopyRange ? "copy kernel: entry out of range (skipped)"
                      : "hash kernel: tile out of range (skipped)";
        return flag == kErrBulkTimeout ? EAKV_E_TIMEOUT : EAKV_E_RANGE;
    }
    return EAKV_OK;
}

int eakv_selfcheck_limits(eakv_ctx* ctx, int64_t gpu_blocks, int64_t tier_slots, int64_t hash_blocks) {
    if (!ctx || ctx->device < 0) return EAKV_E_INVAL;
    if (gpu_blocks < 0 || gpu_blocks > ctx->cfg.gpu_blocks || tier_slots < 0 || tier_slots > ctx->tier_slots ||
        hash_blocks < 0)
        return EAKV_E_INVAL;
    ctx->check_gpu_blocks = gpu_blocks ? gpu_blocks : ctx->cfg.gpu_blocks;
    ctx->check_tier_slots = tier_slots ? tier_slots : ctx->tier_slots;
    ctx->check_hash_blocks = hash_blocks;
    return EAKV_OK;
}

int eakv_selfcheck_fail_next_transfer(eakv_ctx* ctx, int32_t code) {
    if (!ctx || code > 0) return EAKV_E_INVAL;
    ctx->fail_next_transfer = code;
    return EAKV_OK;
}

namespace {
// the injected failure of eakv_selfcheck_fail_next_transfer, once
int injected_failure(eakv_ctx* ctx) {
    const int rc = ctx->fail_next_transfer;
    ctx->fail_next_transfer = 0;
    return rc;
}
}  // namespace

int eakv_selfcheck_wait_probe(eakv_ctx* ctx, void* cuda_stream) {
    if (!ctx || ctx->device < 0) return EAKV_E_INVAL;
    DeviceGuard g(ctx->device);
    CU(launch_wait_probe(ctx->d_error_flag, static_cast<cudaStream_t>(cuda_stream)));
    ctx->stats.kernel_launches += 1;
    return EAKV_OK;
}

int eakv_destroy(eakv_ctx* ctx) {
    if (!ctx) return EAKV_E_INVAL;
    if (ctx->device < 0) {
        free_all(ctx);
        return EAKV_OK;
    }
    DeviceGuard g(ctx->device);
    cudaDeviceSynchronize();
    free_all(ctx);
    return EAKV_OK;
}

// ------------------------------------------------------------------------------------------
// hashing
// ------------------------------------------------------------------------------------------
int eakv_hash_blocks(eakv_ctx* ctx, const int32_t* tokens_dev, int64_t n_tokens,
                     uint64_t parent_hash, uint64_t* hashes_dev, int64_t* n_blocks_out,
                     void* cuda_stream) {
    if (!ctx || n_tokens < 0 || ctx->device < 0) return EAKV_E_INVAL;
    const int b = ctx->cfg.block_size;
    const int64_t nblk = n_tokens / b;
    if (n_blocks_out) *n_blocks_out = nblk;
    if (nblk == 0) return EAKV_OK;
    if (!tokens_dev || !hashes_dev) return EAKV_E_INVAL;
    if (((uintptr_t)tokens_dev & 3) || ((uintptr_t)hashes_dev & 7)) return EAKV_E_INVAL;
    DeviceGuard g(ctx->device);
    if (!device_readable(tokens_dev) || !device_readable(hashes_dev)) return EAKV_E_INVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool generic = hash_thread_per_block(b);
    const bool vec = (b % 4) == 0 && (((uintptr_t)tokens_dev & 15) == 0);
    const int tile_blocks = hash_tile_blocks(b, nblk);
    // split at the scratch capacity; a later piece reads its parent from the previous key
    const int64_t cap = ctx->hash_scratch_blocks;
    int64_t done = 0;
    while (done < nblk) {
        const int64_t cur = std::min(cap, nblk - done);
        HashLaunch L;
        L.tokens = tokens_dev + done * b;
        L.keys = hashes_dev + done;
        L.partial = ctx->d_partial;
        L.counters = ctx->d_counters;
        L.pow_table = ctx->d_pow;
        if (b <= 64) hash_fill_limbs(L, ctx->h_pow.data(), b); else L.pow_block = ctx->h_pow[b];
        L.tiles = nullptr;
        L.prompts = nullptr;
        L.single_nblk = cur;
        L.single_parent = parent_hash % P61;
        L.single_parent_ptr = done ? hashes_dev + done - 1 : nullptr;
        L.block_size = b;
        L.tile_blocks = tile_blocks;
        L.stages = hash_stages(b);
        L.n_prompts = 0;
        L.tokens_limit = n_tokens - done * b;
        L.blocks_limit = ctx->check_hash_blocks > 0 ? std::min(cur, ctx->check_hash_blocks) : cur;
        L.error_flag = ctx->d_error_flag;
        const int n_tiles = (int)((cur + tile_blocks - 1) / tile_blocks);
        const bool piece_vec = vec && (((done * b) & 3) == 0);
        cudaError_t e = launch_hash(L, n_tiles, generic, piece_vec, stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "hash kernel launch");
        ctx->stats.kernel_launches += 1;
        done += cur;
    }
    ctx->stats.tokens_hashed += nblk * b;
    return EAKV_OK;
}

int eakv_hash_blocks_batched(eakv_ctx* ctx, const int32_t* tokens_dev,
                             const int64_t* offsets_host, int64_t n_prompts,
                             const uint64_t* parents_host, uint64_t* hashes_dev,
                             int64_t* block_offsets_out, void* cuda_stream) {
    if (!ctx || n_prompts < 0 || !offsets_host || ctx->device < 0) return EAKV_E_INVAL;
    const int b = ctx->cfg.block_size;
    int64_t total_blocks = 0;
    for (int64_t i = 0; i < n_prompts; ++i) {
        if (offsets_host[i + 1] < offsets_host[i] || offsets_host[i] < 0) return EAKV_E_INVAL;
        total_blocks += (offsets_host[i + 1] - offsets_host[i]) / b;
    }
    if (n_prompts > ctx->max_prompts || total_blocks > ctx->hash_scratch_blocks)
        return EAKV_E_CAPACITY;
    if (block_offsets_out) {
        int64_t acc = 0;
        for (int64_t i = 0; i < n_prompts; ++i) {
            block_offsets_out[i] = acc;
            acc += (offsets_host[i + 1] - offsets_host[i]) / b;
        }
        block_offsets_out[n_prompts] = acc;
    }
    if (total_blocks == 0) return EAKV_OK;
    if (!tokens_dev || !hashes_dev) return EAKV_E_INVAL;
    if (((uintptr_t)tokens_dev & 3) || ((uintptr_t)hashes_dev & 7)) return EAKV_E_INVAL;
    DeviceGuard g(ctx->device);
    if (!device_readable(tokens_dev) || !device_readable(hashes_dev)) return EAKV_E_INVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool generic = hash_thread_per_block(b);
    bool vec = (b % 4) == 0 && (((uintptr_t)tokens_dev & 15) == 0);
    const int tile_blocks = hash_tile_blocks(b, total_blocks);

    int64_t n_tiles = 0;
    for (int64_t i = 0; i < n_prompts; ++i) {
        const int64_t nb = (offsets_host[i + 1] - offsets_host[i]) / b;
        n_tiles += (nb + tile_blocks - 1) / tile_blocks;
        if (nb > 0 && (offsets_host[i] & 3)) vec = false;
    }
    const size_t need = (size_t)n_prompts * sizeof(HashPrompt) + (size_t)n_tiles * sizeof(HashTile);
    if (need > ctx->ring_bytes || n_tiles > INT32_MAX) return EAKV_E_CAPACITY;

    RingSlot* s = nullptr;
    int rc = ring_acquire(ctx, &s);
    if (rc != EAKV_OK) return rc;
    HashPrompt* hp = static_cast<HashPrompt*>(s->host);
    HashTile* ht = reinterpret_cast<HashTile*>(hp + n_prompts);
    int64_t acc = 0, t = 0;
    for (int64_t i = 0; i < n_prompts; ++i) {
        const int64_t nb = (offsets_host[i + 1] - offsets_host[i]) / b;
        const int64_t tiles = (nb + tile_blocks - 1) / tile_blocks;
        hp[i].tok_off = offsets_host[i];
        hp[i].blk_off = acc;
        hp[i].nblk = nb;
        hp[i].parent = (parents_host ? parents_host[i] : ctx->seed) % P61;
        hp[i].tiles = (int32_t)tiles;
        hp[i].pad = 0;
        for (int64_t k = 0; k < tiles; ++k) {
            ht[t].prompt = (int32_t)i;
            ht[t].first_block = (int32_t)(k * tile_blocks);
            ++t;
        }
        acc += nb;
    }
    CU(launch_fetch_args(s->dev, s->host, need, stream));
    ctx->stats.kernel_launches += 1;
    HashLaunch L;
    L.tokens = tokens_dev;
    L.keys = hashes_dev;
    L.partial = ctx->d_partial;
    L.counters = ctx->d_counters;
    L.pow_table = ctx->d_pow;
    if (b <= 64) hash_fill_limbs(L, ctx->h_pow.data(), b); else L.pow_block = ctx->h_pow[b];
    L.prompts = static_cast<const HashPrompt*>(s->dev);
    L.tiles = reinterpret_cast<const HashTile*>(L.prompts + n_prompts);
    L.single_nblk = 0;
    L.single_parent = 0;
    L.single_parent_ptr = nullptr;
    L.block_size = b;
    L.tile_blocks = tile_blocks;
    L.stages = hash_stages(b);
    L.n_prompts = (int32_t)n_prompts;
    L.tokens_limit = offsets_host[n_prompts];
    L.blocks_limit = ctx->check_hash_blocks > 0 ? std::min(total_blocks, ctx->check_hash_blocks) : total_blocks;
    L.error_flag = ctx->d_error_flag;
    int launched = 0;
    cudaError_t e = launch_hash(L, (int)n_tiles, generic, vec, stream, &launched);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "hash kernel launch");
    ctx->stats.kernel_launches += launched;
    CU(cudaEventRecord(s->done, stream));
    ctx->stats.tokens_hashed += total_blocks * b;
    return EAKV_OK;
}

// ------------------------------------------------------------------------------------------
// control plane
// ------------------------------------------------------------------------------------------
int eakv_match(const eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks,
               int64_t* gpu_prefix_blocks, int64_t* host_prefix_blocks,
               int32_t* gpu_block_ids_out, int32_t* host_slots_out) {
    if (!ctx || n_blocks < 0 || (n_blocks > 0 && !hashes_host)) return EAKV_E_INVAL;
    int64_t G = 0, H = 0;
    // each walk asks for the table line and the node of the keys 8 and 4 references ahead (hints only)
    for (; G < n_blocks; ++G) {
        if (G + 8 < n_blocks) ctx->gpu_tier->prefetch_table(hashes_host[G + 8]);
        if (G + 4 < n_blocks) ctx->gpu_tier->prefetch_node(hashes_host[G + 4]);
        const int32_t s = ctx->gpu_tier->find(hashes_host[G]);
        if (s < 0) break;
        if (gpu_block_ids_out) gpu_block_ids_out[G] = s;
    }
    for (; H < n_blocks; ++H) {
        if (H + 8 < n_blocks) ctx->host_tier->prefetch_table(hashes_host[H + 8]);
        if (H + 4 < n_blocks) ctx->host_tier->prefetch_node(hashes_host[H + 4]);
        const int32_t s = ctx->host_tier->find(hashes_host[H]);
        if (s < 0) break;
        if (host_slots_out) host_slots_out[H] = s;
    }
    if (gpu_prefix_blocks) *gpu_prefix_blocks = G;
    if (host_prefix_blocks) *host_prefix_blocks = H;
    return EAKV_OK;
}

// decided < 0: the request's first lookup (admission is decided here and the request enters the
// activity and prompt-length windows); 0 / 1: a later lookup of a request whose choice was skip / store
static int tier_step_impl(eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks,
                          int64_t agent_id, int64_t n_tokens, int64_t now_ms, int decided,
                          uint8_t* hit_out, uint8_t* admit_out, int32_t* slot_out,
                          uint64_t* evicted_keys_out, int32_t* evicted_slots_out,
                          int64_t* n_evicted_inout, eakv_step_info* info_out) {
    if (!ctx || n_blocks < 0 || n_tokens < 0) return EAKV_E_INVAL;
    if (n_blocks > 0 && (!hashes_host || !hit_out || !admit_out || !slot_out)) return EAKV_E_INVAL;
    if (n_blocks > ctx->host_tier->capacity()) return EAKV_E_CAPACITY;
    const bool want_evicted = evicted_keys_out || evicted_slots_out;
    if (want_evicted && (!n_evicted_inout || *n_evicted_inout < n_blocks)) return EAKV_E_CAPACITY;

    KeyedLru& T = *ctx->host_tier;
    ctx->adm->publish(now_ms, T.resident());
    // the keys are known ahead of the walk: table line, node and the node's neighbours are asked
    // for 12, 8 and 4 references early (hints only)
    auto hint = [&](int64_t j) {
        if (j + 12 < n_blocks) T.prefetch_table(hashes_host[j + 12]);
        if (j + 8 < n_blocks) T.prefetch_node(hashes_host[j + 8]);
        if (j + 4 < n_blocks) T.prefetch_neighbours(hashes_host[j + 4]);
    };
    for (int64_t j = 0; j < std::min<int64_t>(12, n_blocks); ++j) T.prefetch_table(hashes_host[j]);
    // leading hits: their slots stay valid until the walk reaches the first miss (hits only promote)
    int64_t H = 0;
    for (; H < n_blocks; ++H) {
        hint(H);
        const int32_t s = T.find(hashes_host[H]);
        if (s < 0) break;
        slot_out[H] = s;
    }
    const bool first = decided < 0;
    const bool p = first ? ctx->adm->pressure(agent_id, n_tokens, now_ms, T.resident()) : false;
    const int64_t cb = ctx->chunk_tokens;                 // tokens per tier unit
    const int64_t u = n_tokens / cb - (H * cb) / cb;
    const bool save = first ? !(p && u > ctx->adm->kappa()) : decided != 0;
    eakv_stats& st = ctx->stats;
    if (first) {
        st.requests += 1;
        st.pressure_requests += p;
        st.declined_requests += !save;
    }
    int64_t n_ev = 0;
    for (int64_t j = 0; j < n_blocks; ++j) {
        const uint64_t key = hashes_host[j];
        st.references += 1;
        if (j >= H) hint(j);
        const int32_t s = j < H ? slot_out[j] : T.find(key);
        if (s >= 0) {
            T.promote(s);
            hit_out[j] = 1; admit_out[j] = 0; slot_out[j] = s;
            st.hits += 1;
        } else if (save) {
            bool ev = false;
            uint64_t vkey = 0;
            int32_t vslot = -1;
            const int32_t ns = T.insert(key, &ev, &vkey, &vslot);
            if (ev) {
                if (!ctx->unstored_units.empty()) ctx->unstored_units.erase(vkey);   // a pending write lost its slot
                if (evicted_keys_out) evicted_keys_out[n_ev] = vkey;
                if (evicted_slots_out) evicted_slots_out[n_ev] = vslot;
                ++n_ev;
                ctx->adm->note_eviction(now_ms);
                st.evicted += 1;
            }
            hit_out[j] = 0; admit_out[j] = 1; slot_out[j] = ns;
            st.admitted += 1;
        } else {
            hit_out[j] = 0; admit_out[j] = 0; slot_out[j] = -1;
            st.declined += 1;
        }
    }
    st.resident = T.resident();
    if (n_evicted_inout) *n_evicted_inout = n_ev;
    if (info_out) {
        info_out->host_prefix_blocks = H;
        info_out->new_chunks = u;
        info_out->pressure = p;
        info_out->save = save;
    }
    return EAKV_OK;
}

int eakv_tier_step(eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks,
                   int64_t agent_id, int64_t n_tokens, int64_t now_ms,
                   uint8_t* hit_out, uint8_t* admit_out, int32_t* slot_out,
                   uint64_t* evicted_keys_out, int32_t* evicted_slots_out,
                   int64_t* n_evicted_inout, eakv_step_info* info_out) {
    return tier_step_impl(ctx, hashes_host, n_blocks, agent_id, n_tokens, now_ms, -1, hit_out, admit_out,
                          slot_out, evicted_keys_out, evicted_slots_out, n_evicted_inout, info_out);
}

int eakv_tier_step_again(eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks, int64_t n_tokens,
                         int64_t now_ms, int32_t save, uint8_t* hit_out, uint8_t* admit_out,
                         int32_t* slot_out, uint64_t* evicted_keys_out, int32_t* evicted_slots_out,
                         int64_t* n_evicted_inout, eakv_step_info* info_out) {
    return tier_step_impl(ctx, hashes_host, n_blocks, 0, n_tokens, now_ms, save ? 1 : 0, hit_out, admit_out,
                          slot_out, evicted_keys_out, evicted_slots_out, n_evicted_inout, info_out);
}

int eakv_tier_export(const eakv_ctx* ctx, uint64_t* keys_host_out, int32_t* slots_host_out,
                     int64_t capacity, int64_t* n_out) {
    if (!ctx || !n_out || capacity < 0) return EAKV_E_INVAL;
    *n_out = ctx->host_tier->resident();
    if ((keys_host_out || slots_host_out) && capacity < *n_out) return EAKV_E_CAPACITY;
    ctx->host_tier->export_order(keys_host_out, slots_host_out, capacity);
    return EAKV_OK;
}

int eakv_tier_import(eakv_ctx* ctx, const uint64_t* keys_host, const int32_t* slots_host, int64_t n) {
    if (!ctx || n < 0 || (n > 0 && (!keys_host || !slots_host))) return EAKV_E_INVAL;
    if (!ctx->host_tier->import_order(keys_host, slots_host, n)) return EAKV_E_INVAL;
    ctx->stats.resident = ctx->host_tier->resident();
    return EAKV_OK;
}

int eakv_admission_export(const eakv_ctx* ctx, int64_t* values_host_out, int64_t capacity, int64_t* n_out) {
    if (!ctx || !n_out || capacity < 0) return EAKV_E_INVAL;
    *n_out = ctx->adm->export_state(nullptr, 0);
    if (!values_host_out) return EAKV_OK;
    if (capacity < *n_out) return EAKV_E_CAPACITY;
    ctx->adm->export_state(values_host_out, capacity);
    return EAKV_OK;
}

int eakv_admission_import(eakv_ctx* ctx, const int64_t* values_host, int64_t n) {
    if (!ctx || n <= 0 || !values_host) return EAKV_E_INVAL;
    return ctx->adm->import_state(values_host, n) ? EAKV_OK : EAKV_E_INVAL;
}

int eakv_gpu_tier_step(eakv_ctx* ctx, const uint64_t* hashes_host, int64_t n_blocks,
                       int32_t need_tail, uint8_t* resident_out, int32_t* block_out,
                       int32_t* tail_block_out) {
    if (!ctx || n_blocks < 0) return EAKV_E_INVAL;
    if (n_blocks > 0 && (!hashes_host || !resident_out || !block_out)) return EAKV_E_INVAL;
    if (need_tail && !tail_block_out) return EAKV_E_INVAL;
    KeyedLru& T = *ctx->gpu_tier;
    if (!ctx->held.empty()) return EAKV_E_INVAL;    // running requests hold blocks: use acquire / release
    if (n_blocks + (need_tail ? 1 : 0) + ctx->gpu_unkeyed > T.capacity()) return EAKV_E_CAPACITY;
    bool ev;
    uint64_t vkey;
    int32_t vslot;
    for (int64_t j = 0; j < n_blocks; ++j) {
        const int32_t s = T.find(hashes_host[j]);
        if (s >= 0) {
            T.promote(s);
            resident_out[j] = 1;
            block_out[j] = s;
        } else {
            resident_out[j] = 0;
            block_out[j] = T.insert(hashes_host[j], &ev, &vkey, &vslot);
        }
    }
    if (tail_block_out) *tail_block_out = -1;
    if (need_tail) {
        *tail_block_out = T.take_unkeyed(&ev, &vkey, &vslot);
        ctx->gpu_unkeyed += 1;
    }
    if (ctx->cfg.gpu_free_order == EAKV_FREE_REVERSE)
        for (int64_t j = n_blocks - 1; j >= 0; --j) T.promote(block_out[j]);
    return EAKV_OK;
}

int eakv_gpu_tier_acquire(eakv_ctx* ctx, int64_t request_id, const uint64_t* hashes_host, int64_t n_blocks,
                          int32_t need_tail, uint8_t* resident_out, int32_t* block_out,
                          int32_t* tail_block_out) {
    if (!ctx || n_blocks < 0) return EAKV_E_INVAL;
    if (n_blocks > 0 && (!hashes_host || !resident_out || !block_out)) return EAKV_E_INVAL;
    if (need_tail && !tail_block_out) return EAKV_E_INVAL;
    if (ctx->held.count(request_id)) return EAKV_E_INVAL;
    KeyedLru& T = *ctx->gpu_tier;
    // every key whose block nobody holds yet takes one block out of the free and the evictable
    // ones (a resident one takes itself); blocks held by running requests are out of reach
    int64_t cost = need_tail ? 1 : 0;
    for (int64_t j = 0; j < n_blocks; ++j) {
        const int32_t s = T.find(hashes_host[j]);
        if (s < 0 || !T.is_pinned(s)) ++cost;
    }
    if (n_blocks + (need_tail ? 1 : 0) > T.capacity()) return EAKV_E_CAPACITY;   // never fits
    if (cost > T.free_slots() + T.evictable()) return EAKV_E_BUSY;               // not beside the others
    eakv_ctx::HeldRequest& h = ctx->held[request_id];
    h.blocks.resize((size_t)n_blocks);
    bool ev;
    uint64_t vkey;
    int32_t vslot;
    for (int64_t j = 0; j < n_blocks; ++j) {
        int32_t s = T.find(hashes_host[j]);
        resident_out[j] = s >= 0;
        if (s < 0) s = T.insert(hashes_host[j], &ev, &vkey, &vslot);
        T.pin(s);
        block_out[j] = s;
        h.blocks[(size_t)j] = s;
    }
    if (tail_block_out) *tail_block_out = -1;
    if (need_tail) {
        h.tail = T.take_unkeyed(&ev, &vkey, &vslot);
        *tail_block_out = h.tail;
        ctx->gpu_unkeyed += 1;
    }
    return EAKV_OK;
}

int eakv_gpu_tier_release_request(eakv_ctx* ctx, int64_t request_id) {
    if (!ctx) return EAKV_E_INVAL;
    auto it = ctx->held.find(request_id);
    if (it == ctx->held.end()) return EAKV_E_INVAL;
    KeyedLru& T = *ctx->gpu_tier;
    const std::vector<int32_t>& b = it->second.blocks;
    if (ctx->cfg.gpu_free_order == EAKV_FREE_REVERSE)
        for (size_t j = b.size(); j-- > 0;) T.unpin(b[j]);
    else
        for (size_t j = 0; j < b.size(); ++j) T.unpin(b[j]);
    if (it->second.tail >= 0) {
        T.release_unkeyed(it->second.tail);
        ctx->gpu_unkeyed -= 1;
    }
    ctx->held.erase(it);
    return EAKV_OK;
}

int eakv_gpu_tier_release(eakv_ctx* ctx, int32_t block_id) {
    if (!ctx) return EAKV_E_INVAL;
    if (block_id < 0 || block_id >= ctx->gpu_tier->capacity()) return EAKV_E_RANGE;
    if (!ctx->gpu_tier->is_unkeyed_taken(block_id)) return EAKV_E_INVAL;
    ctx->gpu_tier->release_unkeyed(block_id);
    ctx->gpu_unkeyed -= 1;
    return EAKV_OK;
}

// ------------------------------------------------------------------------------------------
// store / load
// ------------------------------------------------------------------------------------------
int eakv_store(eakv_ctx* ctx, const int32_t* block_table, const uint8_t* admit_mask,
               const int32_t* host_slots, int64_t n_blocks, void* cuda_stream) {
    if (!ctx || n_blocks < 0 || ctx->device < 0) return EAKV_E_INVAL;
    if (n_blocks == 0) return EAKV_OK;
    if (!block_table || !host_slots) return EAKV_E_INVAL;
    // validate and compact before anything is enqueued
    next_epoch(ctx);
    std::vector<int2>& ent = ctx->scratch_entries;
    ent.clear();
    for (int64_t j = 0; j < n_blocks; ++j) {
        if (admit_mask && !admit_mask[j]) continue;
        const int32_t blk = block_table[j], slot = host_slots[j];
        if (blk < 0 || blk >= ctx->cfg.gpu_blocks || slot < 0 || slot >= ctx->tier_slots)
            return EAKV_E_RANGE;
        if (ctx->slot_stamp[slot] == ctx->epoch) return EAKV_E_INVAL;
        ctx->slot_stamp[slot] = ctx->epoch;
        ent.push_back(make_int2(blk, slot));
    }
    const int64_t m = (int64_t)ent.size();
    if (m == 0) return EAKV_OK;
    DeviceGuard g(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = wait_write_behind(ctx, stream);
    if (rc != EAKV_OK) return rc;
    CU(ctx->restores.order_after(ent, stream, true));    // the slots are about to hold other bytes
    rc = move_blocks(ctx, ent, true, stream, 0, ctx->pieces);
    if (rc != EAKV_OK) return rc;
    CU(ctx->stores.enqueued(ent, ctx->tier_slots, stream));
    CU(ctx->block_reads.enqueued(ent, ctx->cfg.gpu_blocks, stream));
    ctx->stats.blocks_stored += m;
    ctx->stats.bytes_stored += m * ctx->block_bytes;
    return EAKV_OK;
}

int eakv_load(eakv_ctx* ctx, const int32_t* host_slots, const int32_t* block_table,
              int64_t n_blocks, void* cuda_stream) {
    if (!ctx || n_blocks < 0 || ctx->device < 0) return EAKV_E_INVAL;
    if (n_blocks == 0) return EAKV_OK;
    if (!block_table || !host_slots) return EAKV_E_INVAL;
    next_epoch(ctx);
    std::vector<int2>& ent = ctx->scratch_entries;
    ent.clear();
    for (int64_t j = 0; j < n_blocks; ++j) {
        const int32_t blk = block_table[j], slot = host_slots[j];
        if (blk < 0 || blk >= ctx->cfg.gpu_blocks || slot < 0 || slot >= ctx->tier_slots)
            return EAKV_E_RANGE;
        if (ctx->blk_stamp[blk] == ctx->epoch) return EAKV_E_INVAL;
        ctx->blk_stamp[blk] = ctx->epoch;
        ent.push_back(make_int2(blk, slot));
    }
    const int64_t m = n_blocks;
    DeviceGuard g(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = EAKV_OK;
    if (ctx->wb_pending) {                        // a slot may still be receiving a deferred write
        bool touches = false;
        for (int64_t j = 0; j < m && !touches; ++j) touches = ctx->wb_slots[ent[j].y] != 0;
        if (touches) rc = wait_write_behind(ctx, stream);
        if (rc != EAKV_OK) return rc;
    }
    CU(ctx->stores.order_after(ent, stream, false));
    CU(ctx->block_reads.order_after(ent, stream, true));   // the blocks are about to hold other bytes
    rc = move_blocks(ctx, ent, false, stream, 0, ctx->pieces);
    if (rc != EAKV_OK) return rc;
    CU(ctx->restores.enqueued(ent, ctx->tier_slots, stream));
    ctx->stats.blocks_loaded += m;
    ctx->stats.bytes_loaded += m * ctx->block_bytes;
    return EAKV_OK;
}

int eakv_load_layers(eakv_ctx* ctx, const int32_t* host_slots, const int32_t* block_table,
                     int64_t n_blocks, int32_t layers_per_group, void* const* events,
                     int32_t n_events, void* cuda_stream) {
    if (!ctx || n_blocks < 0 || ctx->device < 0 || layers_per_group <= 0) return EAKV_E_INVAL;
    const int L = ctx->cfg.num_layers;
    const int groups = (L + layers_per_group - 1) / layers_per_group;
    if (n_events != groups || (groups > 0 && !events)) return EAKV_E_INVAL;
    for (int g = 0; g < groups; ++g)
        if (!events[g]) return EAKV_E_INVAL;
    if (n_blocks > 0 && (!block_table || !host_slots)) return EAKV_E_INVAL;
    next_epoch(ctx);
    std::vector<int2>& ent = ctx->scratch_entries;
    ent.clear();
    for (int64_t j = 0; j < n_blocks; ++j) {
        const int32_t blk = block_table[j], slot = host_slots[j];
        if (blk < 0 || blk >= ctx->cfg.gpu_blocks || slot < 0 || slot >= ctx->tier_slots)
            return EAKV_E_RANGE;
        if (ctx->blk_stamp[blk] == ctx->epoch) return EAKV_E_INVAL;
        ctx->blk_stamp[blk] = ctx->epoch;
        ent.push_back(make_int2(blk, slot));
    }
    DeviceGuard g(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (ctx->wb_pending) {
        bool touches = false;
        for (size_t j = 0; j < ent.size() && !touches; ++j) touches = ctx->wb_slots[ent[j].y] != 0;
        if (touches) {
            const int rcw = wait_write_behind(ctx, stream);
            if (rcw != EAKV_OK) return rcw;
        }
    }
    if (n_blocks > 0) {
        CU(ctx->stores.order_after(ent, stream, false));
        CU(ctx->block_reads.order_after(ent, stream, true));
    }
    for (int grp = 0; grp < groups; ++grp) {
        const int l0 = grp * layers_per_group;
        const int l1 = std::min(L, l0 + layers_per_group);
        if (n_blocks > 0) {
            int rc = move_blocks(ctx, ent, false, stream, 2 * l0, 2 * (l1 - l0));
            if (rc != EAKV_OK) return rc;
        }
        CU(cudaEventRecord(static_cast<cudaEvent_t>(events[grp]), stream));
    }
    if (n_blocks > 0) CU(ctx->restores.enqueued(ent, ctx->tier_slots, stream));
    ctx->stats.blocks_loaded += n_blocks;
    ctx->stats.bytes_loaded += n_blocks * ctx->block_bytes;
    return EAKV_OK;
}

int eakv_store_layers(eakv_ctx* ctx, const int32_t* block_table, const uint8_t* admit_mask,
                      const int32_t* host_slots, int64_t n_blocks, int32_t layers_per_group,
                      void* const* ready_events, int32_t n_events, void* cuda_stream) {
    if (!ctx || n_blocks < 0 || ctx->device < 0 || layers_per_group <= 0) return EAKV_E_INVAL;
    const int L = ctx->cfg.num_layers;
    const int groups = (L + layers_per_group - 1) / layers_per_group;
    if (n_events != groups || (groups > 0 && !ready_events)) return EAKV_E_INVAL;
    if (n_blocks > 0 && (!block_table || !host_slots)) return EAKV_E_INVAL;
    next_epoch(ctx);
    std::vector<int2>& ent = ctx->scratch_entries;
    ent.clear();
    for (int64_t j = 0; j < n_blocks; ++j) {
        if (admit_mask && !admit_mask[j]) continue;
        const int32_t blk = block_table[j], slot = host_slots[j];
        if (blk < 0 || blk >= ctx->cfg.gpu_blocks || slot < 0 || slot >= ctx->tier_slots)
            return EAKV_E_RANGE;
        if (ctx->slot_stamp[slot] == ctx->epoch) return EAKV_E_INVAL;
        ctx->slot_stamp[slot] = ctx->epoch;
        ent.push_back(make_int2(blk, slot));
    }
    const int64_t m = (int64_t)ent.size();
    DeviceGuard g(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (m > 0) {
        int rcw = wait_write_behind(ctx, stream);
        if (rcw != EAKV_OK) return rcw;
        CU(ctx->restores.order_after(ent, stream, true));
    }
    for (int grp = 0; grp < groups; ++grp) {
        const int l0 = grp * layers_per_group;
        const int l1 = std::min(L, l0 + layers_per_group);
        // the group's layers are read only after the producer has said they are complete
        if (ready_events[grp]) CU(cudaStreamWaitEvent(stream, static_cast<cudaEvent_t>(ready_events[grp]), 0));
        if (m > 0) {
            int rc = move_blocks(ctx, ent, true, stream, 2 * l0, 2 * (l1 - l0));
            if (rc != EAKV_OK) return rc;
        }
    }
    if (m > 0) {
        CU(ctx->stores.enqueued(ent, ctx->tier_slots, stream));
        CU(ctx->block_reads.enqueued(ent, ctx->cfg.gpu_blocks, stream));
    }
    ctx->stats.blocks_stored += m;
    ctx->stats.bytes_stored += m * ctx->block_bytes;
    return EAKV_OK;
}

// ------------------------------------------------------------------------------------------
// turns: one at a time (eakv_turn_*), or several running requests at once (eakv_request_*)
// ------------------------------------------------------------------------------------------
namespace {

// Which of the units the turn admitted are still its own to write (owned_u), once per turn.  A
// single turn owns all of them: nothing comes between its begin and its end.  A request owns those
// that no other request's lookup has evicted since its own (the reference model saw this request's
// write at its lookup, so a later eviction simply overwrote it); they leave the pending set here.
void claim_units(eakv_ctx* ctx, TurnState& T) {
    if (T.claimed) return;
    T.claimed = true;
    const uint64_t* ukeys = T.unit_keys.empty() ? T.keys.data() : T.unit_keys.data();
    T.owned_u.assign(T.admit_u.size(), 0);
    for (size_t c = 0; c < T.admit_u.size(); ++c) {
        if (!T.admit_u[c]) continue;
        if (T.request_id == kNoRequest) {
            T.owned_u[c] = 1;
            continue;
        }
        auto it = ctx->unstored_units.find(ukeys[c]);
        if (it != ctx->unstored_units.end() && it->second == T.request_id) {
            T.owned_u[c] = 1;
            ctx->unstored_units.erase(it);
        }
    }
}

// Take back what an open turn registered but will never produce.  host_units: the tier units the
// turn admitted and still owns (claim_units) leave the host index (their slots were never written).
// gpu_mode 1: every GPU
// block the turn newly keyed leaves the GPU index (nothing was restored or computed); 2: only
// those the engine was to fill (the restored ones hold their bytes).  A block another running
// request shares stays.  Promotions and evictions the turn caused stand.  Lets the turn's GPU
// blocks go (pins, tail block).
void withdraw_turn(eakv_ctx* ctx, TurnState& T, bool host_units, int gpu_mode) {
    claim_units(ctx, T);
    if (host_units) {
        int64_t n = 0;
        const uint64_t* ukeys = T.unit_keys.empty() ? T.keys.data() : T.unit_keys.data();
        // last admitted first, so that the free stack hands the slots out again in the same order
        for (size_t c = T.owned_u.size(); c-- > 0;)
            if (T.owned_u[c] && ctx->host_tier->erase(ukeys[c]) >= 0) ++n;
        ctx->stats.admitted -= n;
        ctx->stats.resident = ctx->host_tier->resident();
    }
    if (T.request_id != kNoRequest && ctx->held.count(T.request_id)) {
        // the pins go first (without the tail: it is released below)
        auto it = ctx->held.find(T.request_id);
        it->second.tail = -1;
        eakv_gpu_tier_release_request(ctx, T.request_id);
    }
    if (gpu_mode) {
        for (size_t j = T.block.size(); j-- > 0;) {
            const bool drop = gpu_mode == 1 ? !T.resident[j] : T.fill[j] != 0;
            if (drop) ctx->gpu_tier->erase(T.keys[j]);
        }
    }
    if (T.tail >= 0) {
        eakv_gpu_tier_release(ctx, T.tail);
        T.tail = -1;
    }
    T.open = false;
}

// decided < 0: the request's first lookup; 0 / 1: a later lookup with that store/skip choice
int turn_begin_impl(eakv_ctx* ctx, TurnState& T, int64_t request_id, const int32_t* tokens, int64_t n_tokens,
                    const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms, int decided,
                    void* cuda_stream, eakv_turn_view* view, int32_t layers_per_group = 0,
                    void* const* events = nullptr, int32_t n_events = 0) {
    const bool as_request = request_id != kNoRequest;
    const bool bookkeeping_only = ctx->device < 0;
    if (layers_per_group < 0) return EAKV_E_INVAL;
    if (layers_per_group > 0) {                   // the restore in layer groups: one event per group
        const int groups = (ctx->cfg.num_layers + layers_per_group - 1) / layers_per_group;
        if (n_events != groups || !events) return EAKV_E_INVAL;
        for (int g = 0; g < groups; ++g)
            if (!events[g]) return EAKV_E_INVAL;
    }
    const int b = ctx->cfg.block_size;
    const int64_t R = ctx->chunk_tokens / b;
    const int64_t nblk = n_tokens / b;
    const int64_t nu = nblk / R;
    const bool need_tail = (n_tokens % b) != 0;
    if (n_known > nblk) n_known = nblk;
    // a context without a device cannot hash: the caller supplies every key
    if (bookkeeping_only && n_known < nblk) return EAKV_E_INVAL;
    if (nblk > n_known && !tokens) return EAKV_E_INVAL;
    if (nblk > n_known && !bookkeeping_only && !device_readable(tokens)) return EAKV_E_INVAL;   // (ordinary host memory)
    // everything that can be refused without a CUDA error is refused here, before either tier changes
    if (nu > ctx->host_tier->capacity()) return EAKV_E_CAPACITY;
    if (!as_request && nblk + (need_tail ? 1 : 0) + ctx->gpu_unkeyed > ctx->gpu_tier->capacity())
        return EAKV_E_CAPACITY;
    DeviceGuard g(bookkeeping_only ? -1 : ctx->device);
    T.keys.resize((size_t)nblk);
    uint64_t* keys = T.keys.data();
    if (n_known > 0) std::memcpy(keys, known_keys, (size_t)n_known * 8);
    if (nblk > n_known) {
        // hash into mapped pinned memory (grown in powers of two), then keep a copy with the turn
        const int64_t need = nblk - n_known;
        if (need > ctx->turn_keys_cap) {
            int64_t cap = 4096;
            while (cap < need) cap <<= 1;
            if (ctx->turn_keys) {
                CU(cudaStreamSynchronize(ctx->lookup_stream));
                CU(cudaFreeHost(ctx->turn_keys));
                ctx->turn_keys = nullptr;
                ctx->turn_keys_cap = 0;
            }
            cudaError_t e = cudaHostAlloc(&ctx->turn_keys, (size_t)cap * 8,
                                          cudaHostAllocMapped | cudaHostAllocPortable);
            if (e != cudaSuccess) {
                cudaGetLastError();
                return EAKV_E_NOMEM;
            }
            ctx->turn_keys_cap = cap;
        }
        if (!ctx->lookup_stream) CU(cudaStreamCreateWithFlags(&ctx->lookup_stream, cudaStreamNonBlocking));
        const uint64_t parent = n_known ? keys[n_known - 1] : ctx->seed;
        int rc = eakv_hash_blocks(ctx, tokens + n_known * b, need * (int64_t)b, parent, ctx->turn_keys, nullptr,
                                  ctx->lookup_stream);
        if (rc != EAKV_OK) return rc;
        CU(cudaStreamSynchronize(ctx->lookup_stream));
        std::memcpy(keys + n_known, ctx->turn_keys, (size_t)need * 8);
    }
    // tier units: one key per full chunk (the key at the chunk's last block)
    const uint64_t* ukeys = keys;
    T.unit_keys.clear();
    if (R > 1) {
        T.unit_keys.resize((size_t)nu);
        for (int64_t c = 0; c < nu; ++c) T.unit_keys[c] = keys[c * R + R - 1];
        ukeys = T.unit_keys.data();
    }
    T.block.resize((size_t)nblk); T.resident.resize((size_t)nblk);
    T.fill.assign((size_t)nblk, 0);
    T.hit.resize((size_t)nu); T.admit_u.assign((size_t)nu, 0); T.slot_u.resize((size_t)nu);
    T.evicted_keys.resize((size_t)nu); T.evicted_slots.resize((size_t)nu);
    T.host_slots.resize((size_t)nu);
    T.request_id = request_id;
    T.tail = -1;
    T.stored = false;
    T.claimed = false;
    T.owned_u.clear();
    // The GPU side first -- a running request whose blocks do not fit beside the others is refused
    // here with both tiers untouched -- then the host tier.  Each walk also answers the lookup: up to
    // its first miss a walk only promotes, so the leading run of keys it found resident is the
    // longest cached prefix as it stood before the turn (G; H with the slots of those units).
    int32_t tail = -1;
    int rc;
    if (as_request)
        rc = eakv_gpu_tier_acquire(ctx, request_id, keys, nblk, need_tail, T.resident.data(), T.block.data(), &tail);
    else
        rc = eakv_gpu_tier_step(ctx, keys, nblk, need_tail, T.resident.data(), T.block.data(), &tail);
    if (rc != EAKV_OK) return rc;
    int64_t G = 0;
    while (G < nblk && T.resident[G]) ++G;
    // a unit that another open request admitted but has not stored yet cannot be restored (read
    // before this turn's own admissions join that set)
    int64_t pending_from = nu;
    if (!ctx->unstored_units.empty())
        for (int64_t c = 0; c < nu; ++c)
            if (ctx->unstored_units.count(ukeys[c])) { pending_from = c; break; }
    T.tail = tail;
    T.open = true;
    int64_t n_ev = nu;
    eakv_step_info info;
    rc = tier_step_impl(ctx, ukeys, nu, agent_id, n_tokens, now_ms, decided, T.hit.data(), T.admit_u.data(),
                        T.slot_u.data(), T.evicted_keys.data(), T.evicted_slots.data(), &n_ev, &info);
    if (rc != EAKV_OK) {                          // (its capacity was checked above)
        withdraw_turn(ctx, T, false, 1);
        return rc;
    }
    int64_t Hu = std::min<int64_t>(info.host_prefix_blocks, pending_from);
    for (int64_t c = 0; c < Hu; ++c) T.host_slots[c] = T.slot_u[c];
    // the units this request admitted are its own to write until another lookup evicts them (before
    // anything below can fail: a withdrawal takes back what is registered here)
    if (as_request)
        for (int64_t c = 0; c < nu; ++c)
            if (T.admit_u[c]) ctx->unstored_units[ukeys[c]] = request_id;
    if (!bookkeeping_only) {
        // blocks this turn will overwrite (restore or the engine's fill, both behind cuda_stream) may
        // still be read by a store that another stream carries: cuda_stream waits for it
        std::vector<int2>& nw = ctx->scratch_entries;
        nw.clear();
        if (tail >= 0) nw.push_back(make_int2(tail, 0));
        for (int64_t j = 0; j < nblk; ++j)
            if (!T.resident[j]) nw.push_back(make_int2(T.block[j], 0));
        const cudaError_t eo = ctx->block_reads.order_after(nw, static_cast<cudaStream_t>(cuda_stream), true);
        if (eo != cudaSuccess) {
            withdraw_turn(ctx, T, true, 1);
            return cuda_fail(ctx, eo, "ordering behind a store that still reads the turn's blocks");
        }
    }
    if (ctx->wb_pending) {
        bool reused = tail >= 0 && ctx->wb_blocks[tail];
        for (int64_t j = 0; j < nblk && !reused; ++j)
            reused = !T.resident[j] && ctx->wb_blocks[T.block[j]];
        if (reused) {
            // the caller is about to overwrite a block the deferred write still reads
            rc = wait_write_behind(ctx, static_cast<cudaStream_t>(cuda_stream));
            if (rc != EAKV_OK) {
                withdraw_turn(ctx, T, true, 1);
                return rc;
            }
            // (the marks stay until the write is seen complete: another stream may come next)
        }
    }
    const int64_t H = Hu * R;
    const int64_t cover = std::max(G, H);
    const int64_t lo = G, hi = H > G ? H : G;
    if (hi > lo || (layers_per_group > 0 && !bookkeeping_only)) {
        // block slots of the restored blocks: chunk slot * R + position inside the chunk
        std::vector<int32_t> slots((size_t)(hi - lo));
        for (int64_t j = lo; j < hi; ++j)
            slots[j - lo] = (int32_t)((int64_t)T.host_slots[j / R] * R + j % R);
        rc = hi > lo ? injected_failure(ctx) : EAKV_OK;
        if (rc == EAKV_OK && !bookkeeping_only) {
            if (layers_per_group > 0)      // (with nothing to restore the events are recorded all the same)
                rc = eakv_load_layers(ctx, slots.data(), T.block.data() + lo, hi - lo, layers_per_group, events,
                                      n_events, cuda_stream);
            else
                rc = eakv_load(ctx, slots.data(), T.block.data() + lo, hi - lo, cuda_stream);
        }
        if (rc != EAKV_OK) {
            // nothing of this turn was restored or will be computed: neither tier may list it
            withdraw_turn(ctx, T, true, 1);
            return rc;
        }
    }
    int64_t n_fill = 0;
    for (int64_t j = cover; j < nblk; ++j)
        if (!T.resident[j]) { T.fill[j] = 1; ++n_fill; }
    // per-block view of the unit decisions, for the store
    T.admit_b.assign((size_t)nblk, 0);
    T.slot_b.assign((size_t)nblk, -1);
    int64_t n_store = 0;
    for (int64_t c = 0; c < nu; ++c) {
        if (!T.admit_u[c]) continue;
        for (int64_t i = 0; i < R; ++i) {
            T.admit_b[c * R + i] = 1;
            T.slot_b[c * R + i] = (int32_t)((int64_t)T.slot_u[c] * R + i);
            ++n_store;
        }
    }
    view->n_blocks = nblk; view->n_units = nu;
    view->gpu_prefix_blocks = G; view->host_prefix_blocks = H;
    view->restore_lo = lo; view->restore_hi = hi;
    view->fresh_tokens = n_tokens - cover * b;
    view->new_chunks = info.new_chunks;
    view->n_fill = n_fill; view->n_stored_blocks = n_store; view->n_evicted = n_ev;
    view->pressure = info.pressure; view->save = info.save; view->tail_block = tail; view->reserved = 0;
    view->keys = keys;
    view->gpu_block = T.block.data(); view->gpu_resident = T.resident.data();
    view->needs_fill = T.fill.data();
    view->hit = T.hit.data(); view->admit = T.admit_u.data(); view->slot = T.slot_u.data();
    view->evicted_keys = T.evicted_keys.data(); view->evicted_slots = T.evicted_slots.data();
    return EAKV_OK;
}

// the store of an open turn's admitted blocks (directly, or deferred on the context's stream);
// layers_per_group > 0: in layer groups behind the producer's events (eakv_store_layers)
int turn_store_impl(eakv_ctx* ctx, TurnState& T, void* cuda_stream, int32_t layers_per_group = 0,
                    void* const* ready_events = nullptr, int32_t n_events = 0) {
    if (layers_per_group < 0) return EAKV_E_INVAL;
    if (layers_per_group > 0) {      // refused before the turn counts as stored
        const int groups = (ctx->cfg.num_layers + layers_per_group - 1) / layers_per_group;
        if (n_events != groups || !ready_events) return EAKV_E_INVAL;
    }
    auto write = [&](void* on_stream) {
        const int64_t n = (int64_t)T.block.size();
        if (layers_per_group > 0)
            return eakv_store_layers(ctx, T.block.data(), T.admit_b.data(), T.slot_b.data(), n, layers_per_group,
                                     ready_events, n_events, on_stream);
        return eakv_store(ctx, T.block.data(), T.admit_b.data(), T.slot_b.data(), n, on_stream);
    };
    const int64_t nblk = (int64_t)T.block.size();
    T.stored = true;
    claim_units(ctx, T);                                     // from here on a stream-ordered restore finds the bytes
    // a unit that another request's lookup evicted in the meantime is not written: its slot is not
    // this request's any more
    const int64_t R = ctx->chunk_tokens / ctx->cfg.block_size;
    for (size_t c = 0; c < T.admit_u.size(); ++c)
        if (T.admit_u[c] && !T.owned_u[c])
            for (int64_t i = 0; i < R; ++i) T.admit_b[c * R + i] = 0;
    bool any_store = false;
    for (int64_t j = 0; j < nblk && !any_store; ++j) any_store = T.admit_b[j] != 0;
    if (!any_store) return EAKV_OK;                          // nothing to write
    if (const int inj = injected_failure(ctx)) return inj;
    if (ctx->device < 0) return EAKV_OK;                     // bookkeeping only
    if (!ctx->cfg.write_behind) return write(cuda_stream);
    // deferred write: on the context's stream, after what precedes it on the caller's stream
    DeviceGuard g(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (!ctx->wb_stream) {
        CU(cudaStreamCreateWithFlags(&ctx->wb_stream, cudaStreamNonBlocking));
        CU(cudaEventCreateWithFlags(&ctx->wb_fence, cudaEventDisableTiming));
        CU(cudaEventCreateWithFlags(&ctx->wb_done, cudaEventDisableTiming));
        ctx->wb_blocks.assign((size_t)ctx->cfg.gpu_blocks, 0);
        ctx->wb_slots.assign((size_t)ctx->tier_slots, 0);
    }
    CU(cudaEventRecord(ctx->wb_fence, stream));
    CU(cudaStreamWaitEvent(ctx->wb_stream, ctx->wb_fence, 0));
    int r = write(ctx->wb_stream);
    if (r != EAKV_OK) return r;
    CU(cudaEventRecord(ctx->wb_done, ctx->wb_stream));
    for (int64_t j = 0; j < nblk; ++j)
        if (T.admit_b[j]) {
            ctx->wb_blocks[T.block[j]] = 1;
            ctx->wb_slots[T.slot_b[j]] = 1;
        }
    ctx->wb_pending = true;
    return EAKV_OK;
}

}  // namespace

int eakv_turn_begin(eakv_ctx* ctx, const int32_t* tokens, int64_t n_tokens,
                    const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                    void* cuda_stream, eakv_turn_view* view) {
    return eakv_turn_begin_layers(ctx, tokens, n_tokens, known_keys, n_known, agent_id, now_ms, 0, nullptr, 0,
                                  cuda_stream, view);
}

int eakv_turn_begin_layers(eakv_ctx* ctx, const int32_t* tokens, int64_t n_tokens,
                           const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                           int32_t layers_per_group, void* const* events, int32_t n_events,
                           void* cuda_stream, eakv_turn_view* view) {
    if (!ctx || !view || n_tokens < 0 || n_known < 0) return EAKV_E_INVAL;
    if (ctx->turn.open || !ctx->held.empty()) return EAKV_E_INVAL;
    if (n_known > 0 && !known_keys) return EAKV_E_INVAL;
    return turn_begin_impl(ctx, ctx->turn, kNoRequest, tokens, n_tokens, known_keys, n_known, agent_id, now_ms,
                           -1, cuda_stream, view, layers_per_group, events, n_events);
}

int eakv_turn_end(eakv_ctx* ctx, void* cuda_stream) {
    return eakv_turn_end_layers(ctx, 0, nullptr, 0, cuda_stream);
}

int eakv_turn_end_layers(eakv_ctx* ctx, int32_t layers_per_group, void* const* ready_events, int32_t n_events,
                         void* cuda_stream) {
    if (!ctx || !ctx->turn.open) return EAKV_E_INVAL;
    const int rc = turn_store_impl(ctx, ctx->turn, cuda_stream, layers_per_group, ready_events, n_events);
    if (rc == EAKV_E_INVAL && !ctx->turn.stored) return rc;                   // bad arguments: the turn stays open
    // a store that could not be enqueued leaves slots unwritten: their keys must not stay listed
    withdraw_turn(ctx, ctx->turn, rc != EAKV_OK, 0);
    return rc;
}

int eakv_turn_abort(eakv_ctx* ctx) {
    if (!ctx || !ctx->turn.open) return EAKV_E_INVAL;
    withdraw_turn(ctx, ctx->turn, true, 2);
    return EAKV_OK;
}

int eakv_request_begin(eakv_ctx* ctx, int64_t request_id, const int32_t* tokens, int64_t n_tokens,
                       const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                       int32_t decided, void* cuda_stream, eakv_turn_view* view) {
    return eakv_request_begin_layers(ctx, request_id, tokens, n_tokens, known_keys, n_known, agent_id, now_ms,
                                     decided, 0, nullptr, 0, cuda_stream, view);
}

int eakv_request_begin_layers(eakv_ctx* ctx, int64_t request_id, const int32_t* tokens, int64_t n_tokens,
                              const uint64_t* known_keys, int64_t n_known, int64_t agent_id, int64_t now_ms,
                              int32_t decided, int32_t layers_per_group, void* const* events, int32_t n_events,
                              void* cuda_stream, eakv_turn_view* view) {
    if (!ctx || !view || n_tokens < 0 || n_known < 0 || request_id == kNoRequest) return EAKV_E_INVAL;
    if (ctx->turn.open || ctx->requests.count(request_id) || ctx->held.count(request_id)) return EAKV_E_INVAL;
    if (n_known > 0 && !known_keys) return EAKV_E_INVAL;
    TurnState& T = ctx->requests[request_id];
    const int rc = turn_begin_impl(ctx, T, request_id, tokens, n_tokens, known_keys, n_known, agent_id, now_ms,
                                   decided < 0 ? -1 : (decided ? 1 : 0), cuda_stream, view, layers_per_group,
                                   events, n_events);
    if (rc != EAKV_OK) ctx->requests.erase(request_id);
    return rc;
}

int eakv_request_store(eakv_ctx* ctx, int64_t request_id, void* cuda_stream) {
    return eakv_request_store_layers(ctx, request_id, 0, nullptr, 0, cuda_stream);
}

int eakv_request_store_layers(eakv_ctx* ctx, int64_t request_id, int32_t layers_per_group,
                              void* const* ready_events, int32_t n_events, void* cuda_stream) {
    if (!ctx) return EAKV_E_INVAL;
    auto it = ctx->requests.find(request_id);
    if (it == ctx->requests.end() || it->second.stored) return EAKV_E_INVAL;
    const int rc = turn_store_impl(ctx, it->second, cuda_stream, layers_per_group, ready_events, n_events);
    if (rc == EAKV_E_INVAL && !it->second.stored) return rc;                  // bad arguments: the request stays open
    if (rc != EAKV_OK) {
        withdraw_turn(ctx, it->second, true, 0);
        ctx->requests.erase(it);
    }
    return rc;
}

int eakv_request_release(eakv_ctx* ctx, int64_t request_id) {
    if (!ctx) return EAKV_E_INVAL;
    auto it = ctx->requests.find(request_id);
    if (it == ctx->requests.end()) return EAKV_E_INVAL;
    // released before its store: the engine never produced the KV, so what was registered is taken back
    if (!it->second.stored) withdraw_turn(ctx, it->second, true, 2);
    else withdraw_turn(ctx, it->second, false, 0);
    ctx->requests.erase(it);
    return EAKV_OK;
}

// ------------------------------------------------------------------------------------------
int eakv_get_stats(const eakv_ctx* ctx, eakv_stats* out) {
    if (!ctx || !out) return EAKV_E_INVAL;
    *out = ctx->stats;
    out->resident = ctx->host_tier->resident();
    return EAKV_OK;
}

void* eakv_tier_ptr(const eakv_ctx* ctx) { return ctx ? ctx->tier : nullptr; }
uint64_t eakv_hash_seed(const eakv_ctx* ctx) { return ctx ? ctx->seed : 0; }
uint64_t eakv_hash_base(const eakv_ctx* ctx) { return ctx ? ctx->base : 0; }

const char* eakv_strerror(int code) {
    switch (code) {
        case EAKV_OK: return "ok";
        case EAKV_E_INVAL: return "invalid argument";
        case EAKV_E_RANGE: return "block id or slot out of range";
        case EAKV_E_CAPACITY: return "request exceeds a capacity";
        case EAKV_E_NOMEM: return "out of memory";
        case EAKV_E_CUDA: return "CUDA runtime error";
        case EAKV_E_TIMEOUT: return "device-side wait timed out";
        case EAKV_E_BUSY: return "GPU blocks held by running requests leave no room";
        default: return "unknown error";
    }
}

const char* eakv_last_cuda_error(const eakv_ctx* ctx) { return ctx ? ctx->cuda_err.c_str() : ""; }

}  // extern "C"
