// Gather / scatter of KV blocks between the paged pool and a slot-major tier.
//
// The pool is 2L independent arrays of pieces ([gpu_blocks][piece_bytes]); a tier slot is
// the 2L pieces of one block back to back.  A work item is (entry j, piece q, 16-KiB
// sub-range); consecutive items walk a slot contiguously, so the tier side streams while
// the pool side jumps one piece at a time.  Nothing is reused: streaming cache hints.
//
// Vector path: a CTA takes one item per loop trip; each thread issues kCopyUnroll
// independent 16-byte loads before its stores, so a full grid keeps >100 KiB per SM in
// flight.  The same kernel serves an HBM tier (HBM roofline), a mapped pinned tier
// (zero-copy over the host link; run it with few CTAs) and the HBM staging buffers of the
// copy-engine strategy.
#include "eakv_internal.h"

#include <cstdlib>

namespace eakv {

template <bool TO_TIER>
__global__ void __launch_bounds__(kCopyThreads, 8)
copy_blocks_vector_kernel(CopyLaunch L) {
    const int64_t items_per_entry = (int64_t)L.pieces * L.subs_per_piece;
    const int64_t n_items = L.n_entries * items_per_entry;
    const int units_per_piece = (int)(L.piece_bytes >> 4);
    for (int64_t it = blockIdx.x; it < n_items; it += gridDim.x) {
        const int64_t j = it / items_per_entry;
        const int r = (int)(it - j * items_per_entry);
        const int q = r / L.subs_per_piece;
        const int sub = r - q * L.subs_per_piece;
        const int2 e = L.entries ? __ldg(L.entries + j) : L.inline_entries[j];
        char* pool = reinterpret_cast<char*>(__ldg(reinterpret_cast<const unsigned long long*>(L.kv_base) + L.q_first + q)) + (int64_t)e.x * L.piece_bytes;
        const int64_t slot = L.slot_from_index ? j : (int64_t)e.y;
        if ((uint64_t)e.x >= (uint64_t)L.gpu_blocks || (uint64_t)slot >= (uint64_t)L.tier_slots) {
            if (threadIdx.x == 0) atomicExch(L.error_flag, kErrCopyRange);
            continue;
        }
        char* tier = L.tier_base + (slot * L.slot_pieces + L.slot_q_first + q) * L.piece_bytes;
        const int4* src = reinterpret_cast<const int4*>(TO_TIER ? pool : tier);
        int4* dst = reinterpret_cast<int4*>(TO_TIER ? tier : pool);
        const int unit0 = sub * (kCopyThreads * kCopyUnroll) + threadIdx.x;
        int4 v[kCopyUnroll];
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u) {
            const int unit = unit0 + u * kCopyThreads;
            if (unit < units_per_piece) v[u] = __ldcs(src + unit);
        }
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u) {
            const int unit = unit0 + u * kCopyThreads;
            if (unit < units_per_piece) __stcs(dst + unit, v[u]);
        }
    }
}

// Argument fetch: per-call arguments (block/slot pairs, hash descriptors) are written by the
// host into mapped pinned memory and pulled into device memory by this kernel instead of a
// copy-engine transfer.  A small host-to-device memcpy would queue on the same copy engine as
// the bulk restores of other requests and wait for all of them (measured: a 32 KB argument
// upload behind a 6 GiB staged restore delayed the store that needed it by the whole restore).
__global__ void fetch_args_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int n16) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x)
        dst[i] = __ldcs(src + i);
}

cudaError_t launch_fetch_args(void* dst_dev, const void* src_host_mapped, size_t bytes,
                              cudaStream_t stream) {
    const int n16 = (int)((bytes + 15) / 16);
    if (n16 <= 0) return cudaSuccess;
    int ctas = (n16 + 255) / 256;
    if (ctas > 64) ctas = 64;
    fetch_args_kernel<<<ctas, 256, 0, stream>>>(static_cast<const uint4*>(src_host_mapped),
                                                static_cast<uint4*>(dst_dev), n16);
    return cudaGetLastError();
}

static int g_vector_ctas_per_sm = 0;

cudaError_t copy_kernels_init() {
    int a = 0, b = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
        &a, copy_blocks_vector_kernel<true>, kCopyThreads, 0);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
        &b, copy_blocks_vector_kernel<false>, kCopyThreads, 0);
    if (e != cudaSuccess) return e;
    g_vector_ctas_per_sm = a < b ? a : b;
    if (g_vector_ctas_per_sm < 1) g_vector_ctas_per_sm = 1;
    return cudaSuccess;
}

int copy_vector_ctas_per_sm() { return g_vector_ctas_per_sm; }

cudaError_t launch_copy_vector(const CopyLaunch& L, bool to_tier, int ctas, cudaStream_t stream) {
    if (L.n_entries <= 0) return cudaSuccess;
    const int64_t n_items = L.n_entries * L.pieces * L.subs_per_piece;
    if (ctas > n_items) ctas = (int)n_items;
    if (ctas < 1) ctas = 1;
    if (to_tier) copy_blocks_vector_kernel<true><<<ctas, kCopyThreads, 0, stream>>>(L);
    else         copy_blocks_vector_kernel<false><<<ctas, kCopyThreads, 0, stream>>>(L);
    return cudaGetLastError();
}

}  // namespace eakv

// ---------------------------------------------------------------------------------------
// Bulk path: one thread per CTA drives a ring of shared-memory stages with 1-D bulk async
// copies (global -> shared completing on an mbarrier, shared -> global in bulk groups).
// Plain per-CTA bulk copies, no tensor maps; every address and size is a multiple of 16 bytes.
// Every wait is bounded: on giving up the thread raises *error_flag, drains what it has
// in flight (bounded again) and returns.
// ---------------------------------------------------------------------------------------
namespace eakv {

constexpr int kBulkMaxStages = 8;
constexpr uint32_t kBulkSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity,
                                                  uint32_t limit = kBulkSpinLimit) {
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if (i > 64) __nanosleep(32);
    }
    return false;
}

struct BulkItem { const char* src; char* dst; uint32_t bytes; };

template <bool TO_TIER>
__device__ __forceinline__ BulkItem bulk_decode(const CopyLaunch& L, int64_t it, int kBulkStageBytes) {
    const int64_t items_per_entry = (int64_t)L.pieces * L.subs_per_piece;
    const int64_t j = it / items_per_entry;
    const int r = (int)(it - j * items_per_entry);
    const int q = r / L.subs_per_piece;
    const int sub = r - q * L.subs_per_piece;
    const int2 e = L.entries ? __ldg(L.entries + j) : L.inline_entries[j];
    const int64_t off = (int64_t)sub * kBulkStageBytes;
    char* pool = reinterpret_cast<char*>(__ldg(reinterpret_cast<const unsigned long long*>(L.kv_base) + L.q_first + q)) +
                 (int64_t)e.x * L.piece_bytes + off;
    const int64_t slot = L.slot_from_index ? j : (int64_t)e.y;
    BulkItem b;
    if ((uint64_t)e.x >= (uint64_t)L.gpu_blocks || (uint64_t)slot >= (uint64_t)L.tier_slots) {
        b.src = nullptr; b.dst = nullptr; b.bytes = 0;      // the caller flags and skips it
        return b;
    }
    char* tier = L.tier_base + (slot * L.slot_pieces + L.slot_q_first + q) * L.piece_bytes + off;
    b.src = TO_TIER ? pool : tier;
    b.dst = TO_TIER ? tier : pool;
    const int64_t left = L.piece_bytes - off;
    b.bytes = (uint32_t)(left < kBulkStageBytes ? left : kBulkStageBytes);
    return b;
}

// Small pieces (at most half a stage): an item is a group of up to L.group_pieces consecutive
// pieces of one block.  They are contiguous on the tier side (one bulk copy) and live in
// separate arrays on the pool side (one bulk copy each), so a stage still carries about
// 16 KiB and the bytes in flight per SM do not shrink with the piece size.
struct BulkGroup { char* tier; int64_t pool_off; int q0; int cnt; };

__device__ __forceinline__ BulkGroup bulk_decode_group(const CopyLaunch& L, int64_t it) {
    const int groups_per_entry = (L.pieces + L.group_pieces - 1) / L.group_pieces;
    const int64_t j = it / groups_per_entry;
    const int g = (int)(it - j * groups_per_entry);
    const int2 e = L.entries ? __ldg(L.entries + j) : L.inline_entries[j];
    const int64_t slot = L.slot_from_index ? j : (int64_t)e.y;
    BulkGroup b;
    b.q0 = g * L.group_pieces;
    b.cnt = L.pieces - b.q0 < L.group_pieces ? L.pieces - b.q0 : L.group_pieces;
    if ((uint64_t)e.x >= (uint64_t)L.gpu_blocks || (uint64_t)slot >= (uint64_t)L.tier_slots) {
        b.tier = nullptr; b.pool_off = 0; b.cnt = 0;        // the caller flags and skips it
        return b;
    }
    b.tier = L.tier_base + (slot * L.slot_pieces + L.slot_q_first + b.q0) * L.piece_bytes;
    b.pool_off = (int64_t)e.x * L.piece_bytes;
    return b;
}

__device__ __forceinline__ char* bulk_pool_piece(const CopyLaunch& L, int q, int64_t pool_off) {
    return reinterpret_cast<char*>(__ldg(reinterpret_cast<const unsigned long long*>(L.kv_base) + L.q_first + q)) + pool_off;
}

template <bool TO_TIER>
__global__ void __launch_bounds__(32)
copy_blocks_bulk_kernel(CopyLaunch L, int kBulkStages, int kBulkStageBytes) {
    int* const error_flag = L.error_flag;
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ __align__(8) uint64_t bars[kBulkMaxStages];
    if (threadIdx.x != 0) return;

    const bool grouped = L.group_pieces > 1;
    const int64_t n_items = grouped ? L.n_entries * ((L.pieces + L.group_pieces - 1) / L.group_pieces)
                                    : L.n_entries * L.pieces * L.subs_per_piece;
    const int64_t first = blockIdx.x, stride = gridDim.x;
    if (first >= n_items) return;
    const int64_t n_my = (n_items - first + stride - 1) / stride;

    for (int s = 0; s < kBulkStages; ++s)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&bars[s])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    auto issue_load = [&](int64_t k) {
        const int s = (int)(k % kBulkStages);
        const uint32_t bar = smem_u32(&bars[s]);
        const uint32_t dst = smem_u32(stage_mem + (size_t)s * kBulkStageBytes);
        if (grouped) {
            const BulkGroup g = bulk_decode_group(L, first + k * stride);
            if (g.cnt == 0) {
                atomicExch(error_flag, kErrCopyRange);
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
                return;
            }
            const uint32_t pb = (uint32_t)L.piece_bytes;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         :: "r"(bar), "r"(pb * g.cnt) : "memory");
            if (TO_TIER) {
                for (int i = 0; i < g.cnt; ++i)
                    asm volatile(
                        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                        :: "r"(dst + i * pb), "l"(bulk_pool_piece(L, g.q0 + i, g.pool_off)), "r"(pb), "r"(bar)
                        : "memory");
            } else {
                asm volatile(
                    "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                    :: "r"(dst), "l"(g.tier), "r"(pb * g.cnt), "r"(bar) : "memory");
            }
            return;
        }
        const BulkItem b = bulk_decode<TO_TIER>(L, first + k * stride, kBulkStageBytes);
        if (b.bytes == 0) {   // self-check tripped: flag it, complete the phase without a copy
            atomicExch(error_flag, kErrCopyRange);
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
            return;
        }
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     :: "r"(bar), "r"(b.bytes) : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
            :: "r"(dst), "l"(b.src), "r"(b.bytes), "r"(bar) : "memory");
    };

    const int64_t prologue = n_my < kBulkStages ? n_my : kBulkStages;
    for (int64_t k = 0; k < prologue; ++k) issue_load(k);
    int64_t loads_issued = prologue;

    bool ok = true;
    int64_t k = 0;
    for (; k < n_my; ++k) {
        const int s = (int)(k % kBulkStages);
        const uint32_t parity = (uint32_t)((k / kBulkStages) & 1);
        if (!mbar_wait_bounded(smem_u32(&bars[s]), parity)) { ok = false; break; }
        const uint32_t src = smem_u32(stage_mem + (size_t)s * kBulkStageBytes);
        if (grouped) {
            const BulkGroup g = bulk_decode_group(L, first + k * stride);
            const uint32_t pb = (uint32_t)L.piece_bytes;
            if (TO_TIER) {
                if (g.cnt != 0)
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                 :: "l"(g.tier), "r"(src), "r"(pb * g.cnt) : "memory");
            } else {
                for (int i = 0; i < g.cnt; ++i)
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                 :: "l"(bulk_pool_piece(L, g.q0 + i, g.pool_off)), "r"(src + i * pb), "r"(pb)
                                 : "memory");
            }
        } else {
            const BulkItem b = bulk_decode<TO_TIER>(L, first + k * stride, kBulkStageBytes);
            if (b.bytes != 0) {
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                             :: "l"(b.dst), "r"(src), "r"(b.bytes) : "memory");
            }
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        if (k >= 1 && loads_issued < n_my) {
            // all but the newest group have finished reading shared memory: stage of item k-1 is free
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            issue_load(loads_issued);
            ++loads_issued;
        }
    }
    if (!ok) {
        atomicExch(error_flag, kErrBulkTimeout);
        // drain the loads still in flight (bounded) so shared memory is quiescent on exit
        for (int64_t d = k + 1; d < loads_issued; ++d) {
            const int s = (int)(d % kBulkStages);
            mbar_wait_bounded(smem_u32(&bars[s]), (uint32_t)((d / kBulkStages) & 1));
        }
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing ever arrives at, with
// a short poll limit, gives up, raises the error word exactly as the copy kernel would and
// returns.  Nothing is in flight, so there is nothing to drain.
__global__ void wait_probe_kernel(int* error_flag, uint32_t limit) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x != 0) return;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_bounded(smem_u32(&bar), 0, limit)) atomicExch(error_flag, kErrBulkTimeout);
}

cudaError_t launch_wait_probe(int* error_flag, cudaStream_t stream) {
    wait_probe_kernel<<<1, 32, 0, stream>>>(error_flag, 1u << 12);
    return cudaGetLastError();
}

// Ring geometry by piece size.  Measured on B200 at full size (6 GiB calls over a 96 GiB pool,
// read+write GB/s): pieces of 16 KiB and more want 3 stages x 16 KiB x 2 CTAs per SM (6,616;
// the small-piece geometry gives 6,379); pieces of 8 KiB and less want more issuing threads
// and about 128 KiB in flight per SM: 2 stages x 8 KiB x 8 CTAs per SM (8 KiB pieces 6,378
// against 6,175; 4 KiB pieces 6,213 against 5,730).  For the large pieces deeper rings or more
// CTAs per SM lose 5-6 %.  (A build with -DEAKV_TUNING reads EAKV_TUNE_BULK_* from the environment for sweeps.)
struct BulkGeometry { int stages, stage_bytes, ctas_per_sm_cap, ctas_per_sm; };
static BulkGeometry g_bulk_geo[2] = {{3, kCopySubBytes, 2, 0}, {2, 8192, 8, 0}};
static bool g_bulk_ready = false;

static cudaError_t bulk_setup() {
    for (BulkGeometry& g : g_bulk_geo) {
#ifdef EAKV_TUNING   // sweep builds only: the shipped library's geometry does not depend on the environment
        if (const char* e = getenv("EAKV_TUNE_BULK_STAGES")) g.stages = atoi(e);
        if (const char* e = getenv("EAKV_TUNE_BULK_STAGE_BYTES")) g.stage_bytes = atoi(e);
        if (const char* e = getenv("EAKV_TUNE_BULK_CTAS_PER_SM")) g.ctas_per_sm_cap = atoi(e);
#endif
        if (g.stages < 2) g.stages = 2;
        if (g.stages > kBulkMaxStages) g.stages = kBulkMaxStages;
        if (g.stage_bytes < 1024 || (g.stage_bytes & 15)) g.stage_bytes = kCopySubBytes;
    }
    size_t smem_max = 0;
    for (const BulkGeometry& g : g_bulk_geo)
        if ((size_t)g.stages * g.stage_bytes > smem_max) smem_max = (size_t)g.stages * g.stage_bytes;
    cudaError_t e = cudaFuncSetAttribute(copy_blocks_bulk_kernel<true>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(copy_blocks_bulk_kernel<false>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e != cudaSuccess) return e;
    for (BulkGeometry& g : g_bulk_geo) {
        int fit = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&fit, copy_blocks_bulk_kernel<true>, 32,
                                                          (size_t)g.stages * g.stage_bytes);
        if (e != cudaSuccess) return e;
        if (fit < 1) fit = 1;
        g.ctas_per_sm = (g.ctas_per_sm_cap >= 1 && g.ctas_per_sm_cap < fit) ? g.ctas_per_sm_cap : fit;
    }
    g_bulk_ready = true;
    return cudaSuccess;
}

// ctas > 0: the caller's explicit grid, used as given; 0: sm_count x this geometry's CTAs per SM
cudaError_t launch_copy_bulk(const CopyLaunch& L_in, bool to_tier, int ctas, int sm_count, cudaStream_t stream) {
    if (L_in.n_entries <= 0) return cudaSuccess;
    if (!g_bulk_ready) {
        cudaError_t e = bulk_setup();
        if (e != cudaSuccess) return e;
    }
    const BulkGeometry& geo = g_bulk_geo[L_in.piece_bytes <= 8192 ? 1 : 0];
    const size_t smem = (size_t)geo.stages * geo.stage_bytes;
    CopyLaunch L = L_in;
    L.subs_per_piece = (int32_t)((L.piece_bytes + geo.stage_bytes - 1) / geo.stage_bytes);
    // pieces of at most half a stage travel in groups that fill the stage (at most 32 per group)
    L.group_pieces = 1;
    if (L.piece_bytes * 2 <= geo.stage_bytes) {
        int64_t g = geo.stage_bytes / L.piece_bytes;
        if (g > 32) g = 32;
        if (g > L.pieces) g = L.pieces;
        L.group_pieces = (int32_t)g;
    }
    if (ctas <= 0) ctas = sm_count * geo.ctas_per_sm;
    const int64_t n_items = L.group_pieces > 1
        ? L.n_entries * ((L.pieces + L.group_pieces - 1) / L.group_pieces)
        : L.n_entries * L.pieces * L.subs_per_piece;
    if (ctas > n_items) ctas = (int)n_items;
    if (ctas < 1) ctas = 1;
    if (to_tier) copy_blocks_bulk_kernel<true><<<ctas, 32, smem, stream>>>(L, geo.stages, geo.stage_bytes);
    else         copy_blocks_bulk_kernel<false><<<ctas, 32, smem, stream>>>(L, geo.stages, geo.stage_bytes);
    return cudaGetLastError();
}

}  // namespace eakv
