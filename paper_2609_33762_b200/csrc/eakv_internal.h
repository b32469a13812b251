// Internal declarations shared by the C-ABI translation unit and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include <cstdlib>

namespace eakv {

// ---- hash ---------------------------------------------------------------------------------
constexpr int kHashThreads = 256;
constexpr int kHashUnroll = 4;
constexpr int kHashTileTokens = kHashThreads * kHashUnroll * 4;   // 4096 tokens per CTA tile
constexpr int kHashMaxBlockSize = 4096;
constexpr int kHashMaxSmem = 80 * 1024;
// staged kernel: limb table + two stages of 256 padded rows at the largest thread-per-block size (64)
constexpr int kHashStagedMaxSmem = 64 * 16 + 2 * kHashThreads * (4 * 64 + 16);

struct HashTile { int32_t prompt; int32_t first_block; };
struct HashPrompt {
    int64_t tok_off;    // first token of the prompt in tokens[]
    int64_t blk_off;    // first key of the prompt in keys[] (and partial[])
    int64_t nblk;       // full blocks
    uint64_t parent;    // h_{-1}
    int32_t tiles;      // CTA tiles covering the prompt
    int32_t pad;
};
struct HashLaunch {
    const int32_t* tokens;
    uint64_t* keys;
    uint64_t* partial;              // scratch: per-block partial sums
    int* counters;                  // scratch: one ticket counter per prompt, zero between launches
    const uint64_t* pow_table;      // B^0 .. B^b
    const HashTile* tiles;          // NULL: single prompt, tile i starts at block i * tile_blocks
    const HashPrompt* prompts;
    int64_t single_nblk;
    uint64_t single_parent;
    const uint64_t* single_parent_ptr;   // non-NULL: read the parent from device memory instead
    int32_t block_size;
    int32_t tile_blocks;
    int32_t stages;                 // sub-tiles in flight per warp (staged kernel 2..4, run kernel 1..2)
    int32_t n_prompts;              // batched launches: prompts described at `prompts`; 0 otherwise
    // B^e for e < 64 as three 21-bit limbs each, passed by value: with the block size known at
    // compile time they become constant-bank operands of the multiply-adds (no load at all)
    uint32_t pw_limbs[3 * 64];
    uint64_t pow_block;             // A = B^b, the per-block multiplier of the scan
    uint64_t apow[5];               // A^0 .. A^4 (the scan launch of the two-launch form)
    // self-check limits: a CTA whose tile would reach past them raises *error_flag and skips
    int64_t tokens_limit;           // tokens readable at `tokens`
    int64_t blocks_limit;           // entries writable at `keys` and `partial`
    int* error_flag;
};
// one thread per block for small or odd block sizes, a group of threads per block otherwise
inline bool hash_thread_per_block(int block_size) { return (block_size % 4) != 0 || block_size <= 64; }
// blocks per CTA tile; large batches get longer tiles so fewer CTAs take tickets
inline int hash_tile_blocks(int block_size, int64_t total_blocks) {
    if (hash_thread_per_block(block_size)) {
#ifdef EAKV_TUNING
        if (const char* e = getenv("EAKV_TUNE_HASH_TILE")) {   // sweep builds only
            const int v = atoi(e);
            if (v >= 1) return v;
        }
#endif
        int t = kHashThreads;
        while (t < 16 * kHashThreads && total_blocks / t > 1184) t *= 2;   // up to a whole 64k-token prompt per CTA
        return t;
    }
    const int t = kHashTileTokens / block_size;
    return t > 1 ? t : 1;
}
// fill L.pw_limbs / L.pow_block from powers B^0 .. B^b held on the host
inline void hash_fill_limbs(HashLaunch& L, const uint64_t* pow_host, int block_size) {
    for (int e = 0; e < 64; ++e) {
        const uint64_t w = e < block_size ? pow_host[e] : 0;
        L.pw_limbs[3 * e + 0] = (uint32_t)(w & 0x1FFFFF);
        L.pw_limbs[3 * e + 1] = (uint32_t)((w >> 21) & 0x1FFFFF);
        L.pw_limbs[3 * e + 2] = (uint32_t)(w >> 42);
    }
    L.pow_block = pow_host[block_size];
    constexpr uint64_t kP61 = (1ull << 61) - 1;
    L.apow[0] = 1;
    for (int q = 1; q < 5; ++q)
        L.apow[q] = (uint64_t)(((unsigned __int128)L.apow[q - 1] * L.pow_block) % kP61);
}
// Sub-tiles in flight per warp in the staged kernel.  Two is the measured optimum: three and
// four (more shared memory, fewer CTAs per SM) were 3-10 % slower.
inline int hash_stages(int block_size) {
#ifdef EAKV_TUNING
    if (const char* e = getenv("EAKV_TUNE_HASH_STAGES")) {      // sweep builds only
        const int v = atoi(e);
        if (v >= 1 && v <= 4 && (size_t)v * kHashThreads * (4 * block_size + 16) <= 136 * 1024) return v;
    }
#endif
    (void)block_size;
    return 2;
}
// also records the current device's SM count for the launch heuristics
cudaError_t hash_kernels_init();
// *launches_out (optional) receives the number of kernels launched: one, or two for large batches
cudaError_t launch_hash(const HashLaunch& L, int n_tiles, bool thread_per_block, bool vec,
                        cudaStream_t stream, int* launches_out = nullptr);

// ---- gather / scatter ---------------------------------------------------------------------
constexpr int kCopyThreads = 256;
constexpr int kCopyUnroll = 4;
constexpr int kCopySubBytes = kCopyThreads * kCopyUnroll * 16;    // 16 KiB per CTA work item

constexpr int kCopyInlineEntries = 32;   // small calls carry their entries in the kernel parameters

struct CopyLaunch {
    const int2* entries;        // {pool block id, tier slot (or staging index)}; NULL: use inline_entries
    int64_t n_entries;
    void* const* kv_base;       // device array of 2L piece-array base pointers
    char* tier_base;            // slot-major destination/source
    int32_t pieces;             // pieces moved per entry (2L, or a layer group's share)
    int32_t q_first;            // first pool piece array of the range moved
    int32_t slot_pieces;        // pieces per slot in the tier-side buffer (2L, or `pieces` for packed staging)
    int32_t slot_q_first;       // where the range starts inside a slot (q_first, or 0 for packed staging)
    int32_t subs_per_piece;     // ceil(piece_bytes / kCopySubBytes)
    int32_t slot_from_index;    // 1: entry j uses slot j (packed staging buffer) instead of entries[j].y
    int32_t group_pieces;       // bulk kernel: consecutive pieces of a block per work item (1: piece by piece)
    int32_t pad0;
    int64_t piece_bytes;
    // self-check limits: an entry outside them raises *error_flag and is skipped
    int64_t gpu_blocks;
    int64_t tier_slots;
    int* error_flag;
    int2 inline_entries[kCopyInlineEntries];
};
// values written to the error flag
constexpr int kErrBulkTimeout = 1, kErrCopyRange = 2, kErrHashRange = 3;
// to_tier: pool -> tier (store/gather); else tier -> pool (load/scatter)
cudaError_t launch_copy_vector(const CopyLaunch& L, bool to_tier, int ctas, cudaStream_t stream);
cudaError_t launch_copy_bulk(const CopyLaunch& L, bool to_tier, int ctas, int sm_count, cudaStream_t stream);
// pull `bytes` (rounded up to 16) of per-call arguments from mapped pinned memory into device memory
cudaError_t launch_fetch_args(void* dst_dev, const void* src_host_mapped, size_t bytes,
                              cudaStream_t stream);
// bounded-wait self-test: a wait that nothing satisfies gives up and raises kErrBulkTimeout
cudaError_t launch_wait_probe(int* error_flag, cudaStream_t stream);
cudaError_t copy_kernels_init();
int copy_vector_ctas_per_sm();

// Can kernels of this process read the address?  Device, managed and registered (pinned) host
// memory: yes.  Ordinary host memory: no -- a kernel given such a pointer takes an illegal-address
// fault that costs the whole CUDA context, so the calls that hand a caller's pointer to a kernel
// ask first and refuse with EAKV_E_INVAL.
inline bool device_readable(const void* p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeHost || at.type == cudaMemoryTypeManaged;
}

}  // namespace eakv
