// Block-key kernel: polynomial prefix hash mod p = 2^61 - 1 over token ids.
//
// h_i = h_{i-1} * B + x_i (x_i = token_i + 1) is a composition of affine maps, and every
// full block contributes the same multiplier A = B^b, so the work splits in two:
//   1. block partials  c_j = sum_k x_{jb+k} * B^{b-1-k} mod p, independent per block:
//      coalesced 16-byte token loads, a 32x61-bit multiply-accumulate per token against a
//      power table in shared memory, lazy reduction once per four tokens.  HBM/ALU bound.
//   2. keys  h_j = h_{j-1} * A + c_j : a scan over affine pairs (a, c) with
//      (a1,c1) o (a2,c2) = (a1 a2, c1 a2 + c2); each thread folds a run of blocks, a
//      warp-level shuffle scan combines threads, shared memory combines warps.
// Both run in one launch: each CTA publishes its tile's partials, takes a ticket on the
// prompt's counter, and the CTA that draws the last ticket of a prompt runs that prompt's
// scan.  No CTA ever waits for another, so there is no spin loop anywhere.
#include "eakv_internal.h"

#ifndef EAKV_HASH_MIN_CTAS
#define EAKV_HASH_MIN_CTAS 1
#endif

namespace eakv {

static constexpr uint64_t P61 = (1ull << 61) - 1;

__device__ __forceinline__ uint64_t reduce_once(uint64_t r) {   // r < 2^63
    r = (r & P61) + (r >> 61);
    if (r >= P61) r -= P61;
    return r;
}

__device__ __forceinline__ uint64_t mulmod61(uint64_t a, uint64_t b) {   // a, b < 2^61
    const uint64_t lo = a * b;
    const uint64_t hi = __umul64hi(a, b);                 // < 2^58
    // 2^61 == 1 (mod p): value = (lo mod 2^61) + (lo >> 61) + hi * 8
    return reduce_once((lo & P61) + ((hi << 3) | (lo >> 61)));
}

// (x * m + add) mod p for a multiplier split once into m0 = low 32 bits, m1 = high 29 bits:
// four 32x32->64 products, no 64-bit high multiply.  x, add < 2^61.
__device__ __forceinline__ uint64_t mulmod61_split_add(uint64_t x, uint32_t m0, uint32_t m1, uint64_t add) {
    const uint32_t x0 = (uint32_t)x, x1 = (uint32_t)(x >> 32);
    const uint64_t p00 = (uint64_t)x0 * m0;                        // < 2^64
    const uint64_t mid = (uint64_t)x0 * m1 + (uint64_t)x1 * m0;    // < 2^62
    const uint64_t p11 = (uint64_t)x1 * m1;                        // < 2^58
    // x*m = p00 + mid * 2^32 + p11 * 2^64, with 2^61 == 1 and 2^64 == 8 (mod p)
    const uint64_t r = (p00 & P61) + (p00 >> 61) + (mid >> 29) + ((mid & ((1ull << 29) - 1)) << 32) +
                       (p11 << 3) + add;                           // < 2^64
    return reduce_once(r);
}

__device__ __forceinline__ uint64_t addmod61(uint64_t a, uint64_t b) {
    uint64_t r = a + b;
    if (r >= P61) r -= P61;
    return r;
}

// sum of four (token+1) * power products, reduced to [0, p)
__device__ __forceinline__ uint64_t dot4(int4 t, const uint64_t* __restrict__ pw, int e_first) {
    // token k of the chunk multiplies B^(e_first - k)
    const uint32_t x[4] = {(uint32_t)t.x + 1u, (uint32_t)t.y + 1u, (uint32_t)t.z + 1u,
                           (uint32_t)t.w + 1u};
    uint64_t s_lo = 0, s_hi = 0;
    uint32_t carry = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint64_t w = pw[e_first - k];
        const uint64_t lo = (uint64_t)x[k] * (uint32_t)w;           // < 2^64
        const uint64_t hi = (uint64_t)x[k] * (uint32_t)(w >> 32);   // < 2^61
        s_lo += lo;
        carry += (s_lo < lo);
        s_hi += hi;                                                 // < 2^63
    }
    // total = s_lo + carry * 2^64 + s_hi * 2^32;  2^64 == 8,  s_hi * 2^32 = (s_hi >> 29) * 2^61 + (s_hi & (2^29-1)) << 32
    uint64_t r = (s_lo & P61) + (s_lo >> 61) + 8ull * carry + (s_hi >> 29) +
                 ((s_hi & ((1ull << 29) - 1)) << 32);               // < 2^63
    return reduce_once(r);
}

struct Pair { uint64_t a, c; };   // h -> h * a + c

__device__ __forceinline__ Pair compose(Pair first, Pair second) {
    Pair r;
    r.a = mulmod61(first.a, second.a);
    r.c = addmod61(mulmod61(first.c, second.a), second.c);
    return r;
}

// Scan of one prompt's block partials into keys, by one whole CTA.
//   partial[0..nblk) -> keys[0..nblk),  keys[j] = keys[j-1] * A + partial[j], keys[-1] = parent
// SHARED: the partials sit in shared memory (a prompt that fits one CTA tile never goes through
// global scratch); otherwise they are read from global memory past L1.
template <bool SHARED>
__device__ __forceinline__ uint64_t load_partial(const uint64_t* p) {
    return SHARED ? *p : __ldcg(p);
}

template <bool SHARED>
__device__ __noinline__ void scan_prompt(const uint64_t* partial, uint64_t* keys, int64_t nblk, uint64_t parent,
                            uint64_t A, Pair* warp_tot /* smem [32] */) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const int64_t per = (nblk + nthr - 1) / nthr;
    const int64_t lo = min((int64_t)tid * per, nblk), hi = min(lo + per, nblk);
    // fold this thread's run (kept in registers when short, so the loads overlap)
    constexpr int kRegRun = 16;
    uint64_t run[kRegRun];
    const bool in_regs = per <= kRegRun;
    if (in_regs) {
#pragma unroll
        for (int i = 0; i < kRegRun; ++i) run[i] = (lo + i < hi) ? load_partial<SHARED>(partial + lo + i) : 0;
    }
    Pair mine{1, 0};
    if (in_regs) {
#pragma unroll
        for (int i = 0; i < kRegRun; ++i) {
            if (lo + i < hi) mine.c = addmod61(mulmod61(mine.c, A), run[i]);
        }
        // the run's multiplier is A^(hi-lo).  All full runs share A^per: one warp-uniform
        // square-and-multiply; only the single ragged run at the end needs its own.
        uint64_t sq = A, a_full = 1;
        for (int64_t n = per; n; n >>= 1) {
            if (n & 1) a_full = mulmod61(a_full, sq);
            sq = mulmod61(sq, sq);
        }
        if (hi - lo == per) {
            mine.a = a_full;
        } else {
            sq = A;
            for (int64_t n = hi - lo; n; n >>= 1) {
                if (n & 1) mine.a = mulmod61(mine.a, sq);
                sq = mulmod61(sq, sq);
            }
        }
    } else {
        for (int64_t j = lo; j < hi; ++j) {
            const uint64_t c = load_partial<SHARED>(partial + j);
            mine.a = mulmod61(mine.a, A);
            mine.c = addmod61(mulmod61(mine.c, A), c);
        }
    }
    // inclusive warp scan over threads (earlier lanes apply first)
    Pair inc = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        Pair up;
        up.a = __shfl_up_sync(0xffffffffu, inc.a, d);
        up.c = __shfl_up_sync(0xffffffffu, inc.c, d);
        if (lane >= d) inc = compose(up, inc);
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        Pair w = lane < nwarp ? warp_tot[lane] : Pair{1, 0};
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            Pair up;
            up.a = __shfl_up_sync(0xffffffffu, w.a, d);
            up.c = __shfl_up_sync(0xffffffffu, w.c, d);
            if (lane >= d) w = compose(up, w);
        }
        warp_tot[lane] = w;   // inclusive over warps
    }
    __syncthreads();
    // exclusive prefix of this thread = (warps before) o (lanes before)
    Pair exc;
    exc.a = __shfl_up_sync(0xffffffffu, inc.a, 1);
    exc.c = __shfl_up_sync(0xffffffffu, inc.c, 1);
    if (lane == 0) exc = Pair{1, 0};
    if (warp > 0) exc = compose(warp_tot[warp - 1], exc);
    uint64_t h = addmod61(mulmod61(parent, exc.a), exc.c);
    if (in_regs) {
#pragma unroll
        for (int i = 0; i < kRegRun; ++i) {
            if (lo + i < hi) {
                h = addmod61(mulmod61(h, A), run[i]);
                keys[lo + i] = h;
            }
        }
    } else {
        for (int64_t j = lo; j < hi; ++j) {
            h = addmod61(mulmod61(h, A), load_partial<SHARED>(partial + j));
            keys[j] = h;
        }
    }
    __syncthreads();
}

// tile = kHashTileChunks 16-byte chunks (or fewer at a prompt's end)
template <bool VEC>
__global__ void __launch_bounds__(kHashThreads)
hash_blocks_kernel(HashLaunch L) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* pw = reinterpret_cast<uint64_t*>(smem_raw);             // [b + 1]
    uint64_t* chunk_sum = pw + L.block_size + 1;                      // [tile chunks]
    __shared__ Pair warp_tot[32];
    __shared__ int is_last;

    const int tid = threadIdx.x;
    for (int e = tid; e <= L.block_size; e += blockDim.x) pw[e] = L.pow_table[e];

    // which prompt and which run of blocks
    int32_t p = 0;
    int64_t first_blk = (int64_t)blockIdx.x * L.tile_blocks;
    int64_t tok0 = 0, blk0 = 0, nblk = L.single_nblk;
    uint64_t parent = L.single_parent;
    int32_t tiles_in_prompt = gridDim.x;
    if (L.tiles != nullptr) {
        const HashTile t = L.tiles[blockIdx.x];
        p = t.prompt;
        first_blk = t.first_block;
        const HashPrompt hp = L.prompts[p];
        tok0 = hp.tok_off; blk0 = hp.blk_off; nblk = hp.nblk; parent = hp.parent;
        tiles_in_prompt = hp.tiles;
    } else if (L.single_parent_ptr != nullptr) {
        parent = *L.single_parent_ptr;
    }
    const int64_t nb_tile = min((int64_t)L.tile_blocks, nblk - first_blk);
    {   // self-check: the tile must lie inside the buffers the caller described
        const int64_t last_blk = blk0 + first_blk + nb_tile;
        const int64_t last_tok = tok0 + (first_blk + nb_tile) * (int64_t)L.block_size;
        if (nb_tile <= 0 || last_blk > L.blocks_limit || last_tok > L.tokens_limit || p < 0) {
            if (threadIdx.x == 0) atomicExch(L.error_flag, kErrHashRange);
            return;
        }
    }
    const int cpb = L.block_size >> 2;                                // chunks per block
    const int n_chunks = (int)nb_tile * cpb;
    const int32_t* tok = L.tokens + tok0 + first_blk * L.block_size;
    __syncthreads();

    // step 1a: per-chunk dot products
    for (int c0 = 0; c0 < n_chunks; c0 += kHashThreads * kHashUnroll) {
        int4 t[kHashUnroll];
#pragma unroll
        for (int u = 0; u < kHashUnroll; ++u) {
            const int c = c0 + u * kHashThreads + tid;
            if (c < n_chunks) {
                if (VEC) {
                    t[u] = __ldcs(reinterpret_cast<const int4*>(tok) + c);
                } else {
                    t[u].x = tok[4 * c]; t[u].y = tok[4 * c + 1];
                    t[u].z = tok[4 * c + 2]; t[u].w = tok[4 * c + 3];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kHashUnroll; ++u) {
            const int c = c0 + u * kHashThreads + tid;
            if (c < n_chunks) {
                const int cib = c % cpb;
                chunk_sum[c] = dot4(t[u], pw, L.block_size - 1 - 4 * cib);
            }
        }
    }
    __syncthreads();
    // step 1b: per-block sums of chunk values -> partials in global scratch
    uint64_t* partial = L.partial + blk0;
    for (int j = tid; j < (int)nb_tile; j += blockDim.x) {
        uint64_t s = 0;
        const uint64_t* cs = chunk_sum + j * cpb;
        for (int k = 0; k < cpb; ++k) s = addmod61(s, cs[k]);
        __stcg(partial + first_blk + j, s);
    }
    // step 2: the CTA that draws the prompt's last ticket scans it
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(L.counters + p, 1);
        is_last = (ticket == tiles_in_prompt - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    scan_prompt<false>(partial, L.keys + blk0, nblk, parent, pw[L.block_size], warp_tot);
    if (tid == 0) L.counters[p] = 0;   // ready for the next launch
}

// Thread-per-block variant: used for small blocks (<= 64 tokens, where it needs the fewest
// instructions per token) and for block sizes that are not a multiple of four.  Each power
// B^e is split into three 21-bit limbs, so a token costs three 32x21-bit multiply-adds into
// three 64-bit sums that cannot overflow for up to 2,048 tokens; the sums are folded mod p
// once per block.  The limb table is read from shared memory (broadcast: all lanes use the
// same power at the same time).  Lanes read 16 bytes at a 4*b-byte stride, so a warp's loads
// together cover a contiguous span that L1 serves.
__device__ __forceinline__ uint64_t fold_limb_sums(uint64_t s0, uint64_t s1, uint64_t s2) {
    // s0 + s1 * 2^21 + s2 * 2^42 (mod p), with 2^61 == 1
    const uint64_t r = (s0 & P61) + (s0 >> 61)
                     + (s1 >> 40) + ((s1 & ((1ull << 40) - 1)) << 21)
                     + (s2 >> 19) + ((s2 & ((1ull << 19) - 1)) << 42);   // < 2^63
    return reduce_once(r);
}

constexpr int kLimbFoldTokens = 1024;   // 1024 * 2^32 * 2^21 = 2^63: no overflow in between

#define EAKV_MAC3(tok, e)                                   \
    do {                                                    \
        const uint32_t x_ = (uint32_t)(tok) + 1u;           \
        const uint4 w_ = pw3[(e)];                          \
        s0 += (uint64_t)x_ * w_.x;                          \
        s1 += (uint64_t)x_ * w_.y;                          \
        s2 += (uint64_t)x_ * w_.z;                          \
    } while (0)

template <bool VEC>
__global__ void __launch_bounds__(kHashThreads)
hash_blocks_tpb_kernel(HashLaunch L) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint4* pw3 = reinterpret_cast<uint4*>(smem_raw);       // limbs of B^0 .. B^(b-1)
    __shared__ Pair warp_tot[32];
    __shared__ int is_last;
    const int tid = threadIdx.x;
    const int b = L.block_size;
    for (int e = tid; e < b; e += blockDim.x) {
        const uint64_t w = L.pow_table[e];
        pw3[e] = make_uint4((uint32_t)(w & 0x1FFFFF), (uint32_t)((w >> 21) & 0x1FFFFF),
                            (uint32_t)(w >> 42), 0u);
    }
    int32_t p = 0;
    int64_t first_blk = (int64_t)blockIdx.x * L.tile_blocks;
    int64_t tok0 = 0, blk0 = 0, nblk = L.single_nblk;
    uint64_t parent = L.single_parent;
    int32_t tiles_in_prompt = gridDim.x;
    if (L.tiles != nullptr) {
        const HashTile t = L.tiles[blockIdx.x];
        p = t.prompt;
        first_blk = t.first_block;
        const HashPrompt hp = L.prompts[p];
        tok0 = hp.tok_off; blk0 = hp.blk_off; nblk = hp.nblk; parent = hp.parent;
        tiles_in_prompt = hp.tiles;
    } else if (L.single_parent_ptr != nullptr) {
        parent = *L.single_parent_ptr;
    }
    const int64_t nb_tile = min((int64_t)L.tile_blocks, nblk - first_blk);
    {   // self-check: the tile must lie inside the buffers the caller described
        const int64_t last_blk = blk0 + first_blk + nb_tile;
        const int64_t last_tok = tok0 + (first_blk + nb_tile) * (int64_t)L.block_size;
        if (nb_tile <= 0 || last_blk > L.blocks_limit || last_tok > L.tokens_limit || p < 0) {
            if (threadIdx.x == 0) atomicExch(L.error_flag, kErrHashRange);
            return;
        }
    }
    __syncthreads();
    uint64_t* partial = L.partial + blk0;
    for (int64_t j = tid; j < nb_tile; j += blockDim.x) {
        const int32_t* t = L.tokens + tok0 + (first_blk + j) * b;
        uint64_t acc = 0;
        for (int k0 = 0; k0 < b; k0 += kLimbFoldTokens) {
            const int k1 = min(b, k0 + kLimbFoldTokens);
            uint64_t s0 = 0, s1 = 0, s2 = 0;
            int k = k0;
            if (VEC) {
                const int4* t4 = reinterpret_cast<const int4*>(t);
#pragma unroll 4
                for (; k + 4 <= k1; k += 4) {
                    const int4 u = __ldg(t4 + (k >> 2));
                    const int e = b - 1 - k;
                    EAKV_MAC3(u.x, e); EAKV_MAC3(u.y, e - 1); EAKV_MAC3(u.z, e - 2); EAKV_MAC3(u.w, e - 3);
                }
            }
            for (; k < k1; ++k) EAKV_MAC3(__ldg(t + k), b - 1 - k);
            acc = addmod61(acc, fold_limb_sums(s0, s1, s2));
        }
        __stcg(partial + first_blk + j, acc);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(L.counters + p, 1);
        is_last = (ticket == tiles_in_prompt - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    scan_prompt<false>(partial, L.keys + blk0, nblk, parent, L.pow_table[b], warp_tot);
    if (tid == 0) L.counters[p] = 0;
}
#undef EAKV_MAC3

// Staged thread-per-block variant for 16-byte-aligned tokens and b % 4 == 0: the tile's
// tokens are brought into shared memory with fully coalesced 16-byte async copies (two
// sub-tiles of 256 blocks in flight), in rows padded by 16 bytes so that the per-thread row
// reads are bank-conflict free; the arithmetic is the same three-limb multiply-add.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(d), "l"(gmem_src) : "memory");
}

#define EAKV_MAC3(tok, e)                                   \
    do {                                                    \
        const uint32_t x_ = (uint32_t)(tok) + 1u;           \
        const uint4 w_ = pw3[(e)];                          \
        s0 += (uint64_t)x_ * w_.x;                          \
        s1 += (uint64_t)x_ * w_.y;                          \
        s2 += (uint64_t)x_ * w_.z;                          \
    } while (0)

// B: the block size when known at compile time (16, 32, 64: loops unroll and every shared-memory
// offset becomes an immediate), 0: read it from the launch descriptor.
// multiply-add against limbs that sit in the kernel parameters (constant bank)
#define EAKV_MACP(tok, e, A0, A1, A2)                              \
    do {                                                           \
        const uint32_t x_ = (uint32_t)(tok) + 1u;                  \
        A0 += (uint64_t)x_ * L.pw_limbs[3 * (e) + 0];              \
        A1 += (uint64_t)x_ * L.pw_limbs[3 * (e) + 1];              \
        A2 += (uint64_t)x_ * L.pw_limbs[3 * (e) + 2];              \
    } while (0)

template <int B>
__global__ void __launch_bounds__(kHashThreads, EAKV_HASH_MIN_CTAS)
hash_blocks_staged_kernel(const __grid_constant__ HashLaunch L) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ Pair warp_tot[32];
    __shared__ int is_last;
    const int tid = threadIdx.x;
    const int b = B ? B : L.block_size, cpb = b >> 2;
    const int row_bytes = 4 * b + 16;
    uint4* pw3 = reinterpret_cast<uint4*>(smem_raw);
    unsigned char* const stage0 = smem_raw + (size_t)b * 16;
    const size_t stage_bytes = (size_t)kHashThreads * row_bytes;
    const int S = L.stages;
    int32_t p = 0;
    int64_t first_blk = (int64_t)blockIdx.x * L.tile_blocks;
    int64_t tok0 = 0, blk0 = 0, nblk = L.single_nblk;
    uint64_t parent = L.single_parent;
    int32_t tiles_in_prompt = gridDim.x;
    if (L.tiles != nullptr) {
        const HashTile t = L.tiles[blockIdx.x];
        p = t.prompt;
        first_blk = t.first_block;
        const HashPrompt hp = L.prompts[p];
        tok0 = hp.tok_off; blk0 = hp.blk_off; nblk = hp.nblk; parent = hp.parent;
        tiles_in_prompt = hp.tiles;
    } else if (L.single_parent_ptr != nullptr) {
        parent = *L.single_parent_ptr;
    }
    const int nb_tile = (int)min((int64_t)L.tile_blocks, nblk - first_blk);
    {   // self-check: the tile must lie inside the buffers the caller described
        const int64_t last_blk = blk0 + first_blk + nb_tile;
        const int64_t last_tok = tok0 + (first_blk + nb_tile) * (int64_t)L.block_size;
        if (nb_tile <= 0 || last_blk > L.blocks_limit || last_tok > L.tokens_limit || p < 0) {
            if (threadIdx.x == 0) atomicExch(L.error_flag, kErrHashRange);
            return;
        }
    }
    const int n_sub = (nb_tile + kHashThreads - 1) / kHashThreads;
    const int4* tile_src = reinterpret_cast<const int4*>(L.tokens + tok0 + first_blk * b);

    // Every warp stages and consumes its own 32 rows, so the main loop needs no block-wide
    // barrier: a warp waits for its own async copies and synchronises only with itself.
    const int lane = tid & 31, warp = tid >> 5;
    auto issue = [&](int r) {
        const int nb = min(kHashThreads, nb_tile - r * kHashThreads);
        const int nb_w = max(0, min(32, nb - warp * 32));
        const int chunks_w = nb_w * cpb;
        const int first_chunk = warp * 32 * cpb;
        const int4* src = tile_src + (size_t)r * kHashThreads * cpb;
        unsigned char* st = stage0 + (r % S) * stage_bytes;
        for (int c = lane; c < chunks_w; c += 32) {
            const int cg = first_chunk + c;
            const int row = cg / cpb, col = cg - row * cpb;
            cp_async16(st + (size_t)row * row_bytes + col * 16, src + cg);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    // exactly one group is committed per sub-tile slot (empty past the end), so "all but the
    // newest S-1 groups are complete" always means that sub-tile r has landed
    for (int r = 0; r < S - 1; ++r) {
        if (r < n_sub) issue(r);
        else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    if (!B) {
        for (int e = tid; e < b; e += blockDim.x) {
            const uint64_t w = L.pow_table[e];
            pw3[e] = make_uint4((uint32_t)(w & 0x1FFFFF), (uint32_t)((w >> 21) & 0x1FFFFF),
                                (uint32_t)(w >> 42), 0u);
        }
        __syncthreads();     // the limb table is shared by the whole CTA
    }
    // A single prompt that fits this one CTA (at most kHashThreads blocks) never leaves the CTA:
    // its partials stay in shared memory and the scan follows after one barrier -- no global
    // scratch, no fence, no ticket.
    __shared__ uint64_t local_partial[kHashThreads];
    const bool lone = L.tiles == nullptr && gridDim.x == 1 && nb_tile <= kHashThreads;
    uint64_t* partial = L.partial + blk0;
    for (int r = 0; r < n_sub; ++r) {
        if (r + S - 1 < n_sub) issue(r + S - 1);
        else asm volatile("cp.async.commit_group;" ::: "memory");
        if (S == 2)      asm volatile("cp.async.wait_group 1;" ::: "memory");
        else if (S == 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
        else             asm volatile("cp.async.wait_group 3;" ::: "memory");
        __syncwarp();
        const int j = r * kHashThreads + tid;
        if (j < nb_tile) {
            const int4* row = reinterpret_cast<const int4*>(stage0 + (r % S) * stage_bytes + (size_t)tid * row_bytes);
            uint64_t acc = 0;
            if (B) {   // b <= 64 < kLimbFoldTokens: one fold per block, fully unrolled
                // two independent accumulator sets: six multiply-add chains in flight
                uint64_t s0 = 0, s1 = 0, s2 = 0, t0 = 0, t1 = 0, t2 = 0;
#pragma unroll
                for (int k = 0; k < (B ? B : 4); k += 4) {
                    const int4 u = row[k >> 2];
                    const int e = (B ? B : 4) - 1 - k;
                    EAKV_MACP(u.x, e, s0, s1, s2); EAKV_MACP(u.y, e - 1, t0, t1, t2);
                    EAKV_MACP(u.z, e - 2, s0, s1, s2); EAKV_MACP(u.w, e - 3, t0, t1, t2);
                }
                acc = fold_limb_sums(s0 + t0, s1 + t1, s2 + t2);
            } else {
                for (int k0 = 0; k0 < b; k0 += kLimbFoldTokens) {
                    const int k1 = min(b, k0 + kLimbFoldTokens);
                    uint64_t s0 = 0, s1 = 0, s2 = 0;
#pragma unroll 4
                    for (int k = k0; k < k1; k += 4) {
                        const int4 u = row[k >> 2];
                        const int e = b - 1 - k;
                        EAKV_MAC3(u.x, e); EAKV_MAC3(u.y, e - 1); EAKV_MAC3(u.z, e - 2); EAKV_MAC3(u.w, e - 3);
                    }
                    acc = addmod61(acc, fold_limb_sums(s0, s1, s2));
                }
            }
            if (lone) local_partial[j] = acc;
            else __stcg(partial + first_blk + j, acc);
        }
        __syncwarp();        // this warp refills the stage S-1 iterations from now
    }
    if (lone) {
        __syncthreads();
        scan_prompt<true>(local_partial, L.keys + blk0, nblk, parent, L.pow_block, warp_tot);
        return;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(L.counters + p, 1);
        is_last = (ticket == tiles_in_prompt - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    scan_prompt<false>(partial, L.keys + blk0, nblk, parent, L.pow_block, warp_tot);
    if (tid == 0) L.counters[p] = 0;
}
#undef EAKV_MAC3

// thread_per_block: see hash_thread_per_block(); vec: 16-byte token loads are allowed
// ---------------------------------------------------------------------------------------
// Run variant for b in {16, 32, 64} and 16-byte-aligned tokens.
//
// A lane owns RUN = 64 / b consecutive blocks (64 tokens, 256 bytes) of a warp tile, so that
// the per-block chain h' = h * A + c over those blocks runs inside the lane, interleaved with
// the next block's multiply-adds, and what the lane publishes per block is already the prefix
// inside its run.  Every warp stages its own tiles (32 lanes x 256 bytes, coalesced 16-byte
// async copies at immediate offsets into rows padded by 16 bytes) in a ring of one or two
// stages and synchronises only with itself; this launch has no fence, ticket or block-wide
// barrier.  A second launch, one CTA per prompt, then needs one modular product per block: it
// scans the run totals (constant multiplier A^RUN), leaves every run's incoming hash in shared
// memory and finishes all blocks with coalesced accesses.  Used for batches of many prompts;
// single prompts keep the one-launch kernels above (a second launch would cost them latency).
//
// Measured on B200, 512 prompts x 65,536 tokens, block 16 (device time of the launches): token
// launch 32 us, of which the loads alone are 29 us and the arithmetic is hidden; scan launch
// 20 us; the one-launch staged kernel takes 64 us for the same work.  Variants that were slower:
// the scan fused behind a ticket (its registers cut the token phase's occupancy: 55-61 us), 512
// threads per scan CTA (22 us), a third launch that applies the incoming hashes (12 + 11 us).
// ---------------------------------------------------------------------------------------
constexpr int kRunThreads = 128;
constexpr int kRunRowBytes = 256 + 16;
constexpr int kRunWarpStage = 32 * kRunRowBytes;                      // 8,704 bytes
constexpr int kRunSmem = 2 * (kRunThreads / 32) * kRunWarpStage;      // 69,632 bytes
constexpr int kRunChunkRuns = 2048;      // runs scanned per pass: their incoming hashes take 16 KiB

template <int RUN>
__device__ __forceinline__ uint64_t pick_pow(const uint64_t (&apow)[5], int m) {
    uint64_t r = apow[RUN];
#pragma unroll
    for (int q = 1; q < RUN; ++q)
        if (m == q) r = apow[q];
    return r;
}

// Shared state of one scan pass.  All full runs have the multiplier M = A^RUN and every thread but
// the last non-empty one holds exactly `per` of them, so the scan over threads needs one modular
// product per step against multipliers that are the same for the whole CTA.
struct ScanShared {
    uint64_t step_pow[5];      // (M^per)^(2^k)
    uint64_t lane_pow[32];     // (M^per)^lane
    uint64_t warp_mult;        // (M^per)^32
    uint64_t warp_tot[32];     // inclusive total of each warp
    uint64_t warp_in[32];      // hash entering each warp
    uint64_t carry;            // hash entering the next pass
};

template <int RUN, int NTHR>
__device__ __forceinline__ void scan_runs(const uint64_t* partial, uint64_t* keys, int64_t nblk, uint64_t parent,
                                          const uint64_t (&apow)[5], uint64_t* h_in, ScanShared* sh) {
    constexpr int kPer = kRunChunkRuns / NTHR;             // runs per thread and pass
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    constexpr int nwarp = NTHR / 32;
    const uint64_t M = apow[RUN];
    // every block a thread finishes has the same position in its run (NTHR is a multiple of RUN)
    const uint64_t my_mult = pick_pow<RUN>(apow, tid % RUN + 1);
    const uint32_t my_m0 = (uint32_t)my_mult, my_m1 = (uint32_t)(my_mult >> 32);
    const uint32_t M0 = (uint32_t)M, M1 = (uint32_t)(M >> 32);
    uint64_t carry = parent;
    for (int64_t base = 0; base < nblk; base += (int64_t)kRunChunkRuns * RUN) {
        const int cblk = (int)min((int64_t)kRunChunkRuns * RUN, nblk - base);
        const int n_runs = (cblk + RUN - 1) / RUN;
        const int m_last = cblk - (n_runs - 1) * RUN;                    // blocks in the pass's last run
        const int per = (n_runs + NTHR - 1) / NTHR;                      // <= kPer
        const int lo = min(tid * per, n_runs), hi = min(lo + per, n_runs);
        if (warp == 0) {          // this pass's uniform multipliers
            uint64_t mper = 1, sq = M;
            for (int n = per; n; n >>= 1) {
                if (n & 1) mper = mulmod61(mper, sq);
                sq = mulmod61(sq, sq);
            }
            uint64_t sp = mper, lp = 1;
#pragma unroll
            for (int k = 0; k < 5; ++k) {
                if (lane == 0) sh->step_pow[k] = sp;
                if ((lane >> k) & 1) lp = mulmod61(lp, sp);
                sp = mulmod61(sp, sp);
            }
            sh->lane_pow[lane] = lp;
            if (lane == 0) sh->warp_mult = sp;
        }
        // all of this thread's run totals at once (a run's total sits at its last block), then Horner
        uint64_t tot[kPer];
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            const int jq = lo + q;
            tot[q] = jq < hi ? __ldcg(partial + base + min((jq + 1) * RUN, cblk) - 1) : 0;
        }
        const bool has_ragged = (hi == n_runs) && (hi > lo) && (m_last != RUN);
        const uint64_t ragged_mult = pick_pow<RUN>(apow, m_last);
        const uint32_t R0 = (uint32_t)ragged_mult, R1 = (uint32_t)(ragged_mult >> 32);
        uint64_t c = 0;
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            if (lo + q < hi) {
                const bool rg = has_ragged && lo + q == hi - 1;
                c = mulmod61_split_add(c, rg ? R0 : M0, rg ? R1 : M1, tot[q]);
            }
        }
        __syncthreads();
        uint64_t inc = c;
#pragma unroll
        for (int k = 0; k < 5; ++k) {
            const uint64_t up = __shfl_up_sync(0xffffffffu, inc, 1 << k);
            if (lane >= (1 << k)) inc = addmod61(mulmod61(up, sh->step_pow[k]), inc);
        }
        uint64_t exc = __shfl_up_sync(0xffffffffu, inc, 1);
        if (lane == 0) exc = 0;
        if (lane == 31) sh->warp_tot[warp] = inc;
        __syncthreads();
        if (tid == 0) {
            uint64_t h = carry;
            for (int w = 0; w < nwarp; ++w) {
                sh->warp_in[w] = h;
                h = addmod61(mulmod61(h, sh->warp_mult), sh->warp_tot[w]);
            }
        }
        __syncthreads();
        uint64_t h = addmod61(mulmod61(sh->warp_in[warp], sh->lane_pow[lane]), exc);
        // incoming hash of each of this thread's runs
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            if (lo + q < hi) {
                h_in[lo + q] = h;
                const bool rg = has_ragged && lo + q == hi - 1;
                h = mulmod61_split_add(h, rg ? R0 : M0, rg ? R1 : M1, tot[q]);
            }
        }
        if (lo < hi && hi == n_runs) sh->carry = h;       // hash at the end of this pass
        __syncthreads();
        carry = sh->carry;
        // key of block i = (incoming hash of its run) * A^(position in run + 1) + prefix inside the run;
        // eight independent blocks per thread and step keep the loads in flight together
        constexpr int kU = 8;
        const uint64_t* pin = partial + base;
        uint64_t* kout = keys + base;
        for (int i0 = tid; i0 < cblk; i0 += NTHR * kU) {
            uint64_t pv[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int i = i0 + u * NTHR;
                pv[u] = i < cblk ? __ldcg(pin + i) : 0;
            }
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int i = i0 + u * NTHR;
                if (i < cblk) kout[i] = mulmod61_split_add(h_in[i / RUN], my_m0, my_m1, pv[u]);
            }
        }
        __syncthreads();
    }
}

template <int B>
__global__ void __launch_bounds__(kRunThreads)
hash_blocks_run_kernel(const __grid_constant__ HashLaunch L) {
    constexpr int RUN = 64 / B;
    constexpr int WT = 32 * RUN;                 // blocks per warp tile
    constexpr int CPB = B / 4;                   // 16-byte chunks per block
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const HashTile tile = L.tiles[blockIdx.x];
    const HashPrompt hp = L.prompts[tile.prompt];
    const int64_t first_blk = tile.first_block;
    const int64_t tok0 = hp.tok_off, blk0 = hp.blk_off, nblk = hp.nblk;
    const int nb_tile = (int)min((int64_t)L.tile_blocks, nblk - first_blk);
    {   // self-check: the tile must lie inside the buffers the caller described
        const int64_t last_blk = blk0 + first_blk + nb_tile;
        const int64_t last_tok = tok0 + (first_blk + nb_tile) * (int64_t)B;
        if (nb_tile <= 0 || last_blk > L.blocks_limit || last_tok > L.tokens_limit || tile.prompt < 0 ||
            (L.tile_blocks % WT) != 0) {
            if (threadIdx.x == 0) atomicExch(L.error_flag, kErrHashRange);
            return;
        }
    }
    const int n_wt = (nb_tile + WT - 1) / WT;
    const int4* tile_src = reinterpret_cast<const int4*>(L.tokens + tok0 + first_blk * B);
    const int S = L.stages;                      // 1: no prefetch (more CTAs per SM), 2: two-stage ring
    unsigned char* const ring = smem_raw + (size_t)warp * S * kRunWarpStage;
    const int dst_lane = (lane >> 4) * kRunRowBytes + (lane & 15) * 16;

    auto issue = [&](int t, int stage) {
        const int nb = min(WT, nb_tile - t * WT);
        const int chunks = nb * CPB;                          // valid 16-byte chunks, 512 when full
        const int4* src = tile_src + (size_t)t * (WT * CPB) + lane;
        unsigned char* dst = ring + stage * kRunWarpStage + dst_lane;
        if (chunks == 512) {
#pragma unroll
            for (int i = 0; i < 16; ++i) cp_async16(dst + i * 2 * kRunRowBytes, src + 32 * i);
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i)
                if (lane + 32 * i < chunks) cp_async16(dst + i * 2 * kRunRowBytes, src + 32 * i);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    const uint64_t A = L.pow_block;
    uint64_t* partial = L.partial + blk0 + first_blk;
    if (S == 2) {
        if (warp < n_wt) issue(warp, 0);
        else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    int it = 0;
    for (int t = warp; t < n_wt; t += kRunThreads / 32, ++it) {
        if (S == 2) {
            // one group per iteration (empty past the end): "all but the newest" = this tile has landed
            if (t + kRunThreads / 32 < n_wt) issue(t + kRunThreads / 32, (it + 1) & 1);
            else asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            issue(t, 0);
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncwarp();
        const unsigned char* row = ring + (S == 2 ? (it & 1) : 0) * kRunWarpStage + lane * kRunRowBytes;
        const int nb = min(WT, nb_tile - t * WT);
        uint64_t chain = 0;
#pragma unroll
        for (int r = 0; r < RUN; ++r) {
            if (lane * RUN + r < nb) {
                const int4* blk = reinterpret_cast<const int4*>(row + r * B * 4);
                uint64_t s0 = 0, s1 = 0, s2 = 0, t0 = 0, t1 = 0, t2 = 0;
#pragma unroll
                for (int k = 0; k < B; k += 4) {
                    const int4 u = blk[k >> 2];
                    const int e = B - 1 - k;
                    EAKV_MACP(u.x, e, s0, s1, s2); EAKV_MACP(u.y, e - 1, t0, t1, t2);
                    EAKV_MACP(u.z, e - 2, s0, s1, s2); EAKV_MACP(u.w, e - 3, t0, t1, t2);
                }
                const uint64_t c = fold_limb_sums(s0 + t0, s1 + t1, s2 + t2);
                chain = r == 0 ? c : addmod61(mulmod61(chain, A), c);
                __stcg(partial + (int64_t)t * WT + lane * RUN + r, chain);
            }
        }
        __syncwarp();        // this warp refills the stage two iterations from now
    }
}

// Second launch: one CTA per prompt turns the run prefixes into keys.
template <int RUN>
__global__ void __launch_bounds__(kRunThreads)
hash_scan_runs_kernel(const __grid_constant__ HashLaunch L) {
    __shared__ ScanShared sh;
    __shared__ __align__(16) uint64_t h_in[kRunChunkRuns];
    const HashPrompt hp = L.prompts[blockIdx.x];
    if (hp.nblk <= 0) return;
    if (hp.blk_off < 0 || hp.blk_off + hp.nblk > L.blocks_limit) {
        if (threadIdx.x == 0) atomicExch(L.error_flag, kErrHashRange);
        return;
    }
    scan_runs<RUN, kRunThreads>(L.partial + hp.blk_off, L.keys + hp.blk_off, hp.nblk, hp.parent, L.apow, h_in, &sh);
}

#undef EAKV_MACP

static int g_hash_sm_count = 148;      // replaced by the device's own count in hash_kernels_init

cudaError_t launch_hash(const HashLaunch& L_in, int n_tiles, bool thread_per_block, bool vec,
                        cudaStream_t stream, int* launches_out) {
    if (launches_out) *launches_out = n_tiles > 0 ? 1 : 0;
    if (n_tiles <= 0) return cudaSuccess;
    HashLaunch L = L_in;
    const bool run_shape = vec && (L.block_size == 16 || L.block_size == 32 || L.block_size == 64);
    if (run_shape && L.stages > 2) L.stages = 2;             // the run kernel has one or two stages
    if (thread_per_block) {
        const size_t smem = (size_t)L.block_size * sizeof(uint4);
        // Many prompts of a block size known at compile time: two launches, the token phase
        // (a lane per run of consecutive blocks) and the per-prompt scan.  Neither needs a fence
        // or a ticket, and the scan's registers do not limit the token phase's occupancy.
#ifdef EAKV_TUNING   // EAKV_TUNE_HASH_KERNEL=staged keeps the single-launch kernel, for A/B runs
        static const bool use_run = [] {
            const char* e = getenv("EAKV_TUNE_HASH_KERNEL");
            return !(e && e[0] == 's');
        }();
#else
        constexpr bool use_run = true;
#endif
        if (run_shape && use_run && L.tiles != nullptr && L.n_prompts > 0 && n_tiles >= 2 * g_hash_sm_count) {
            const size_t rs = L.stages == 2 ? kRunSmem : kRunSmem / 2;
            if (L.block_size == 16)      hash_blocks_run_kernel<16><<<n_tiles, kRunThreads, rs, stream>>>(L);
            else if (L.block_size == 32) hash_blocks_run_kernel<32><<<n_tiles, kRunThreads, rs, stream>>>(L);
            else                         hash_blocks_run_kernel<64><<<n_tiles, kRunThreads, rs, stream>>>(L);
            cudaError_t e = cudaGetLastError();
            if (e != cudaSuccess) return e;
            if (L.block_size == 16)      hash_scan_runs_kernel<4><<<L.n_prompts, kRunThreads, 0, stream>>>(L);
            else if (L.block_size == 32) hash_scan_runs_kernel<2><<<L.n_prompts, kRunThreads, 0, stream>>>(L);
            else                         hash_scan_runs_kernel<1><<<L.n_prompts, kRunThreads, 0, stream>>>(L);
            if (launches_out) *launches_out = 2;
            return cudaGetLastError();
        }
        if (L.stages < 2) L.stages = 2;          // the staged kernel keeps two to four sub-tiles in flight
        const size_t staged = smem + (size_t)L.stages * kHashThreads * (4 * L.block_size + 16);
        if (!vec)                    hash_blocks_tpb_kernel<false><<<n_tiles, kHashThreads, smem, stream>>>(L);
        else if (L.block_size == 16) hash_blocks_staged_kernel<16><<<n_tiles, kHashThreads, staged, stream>>>(L);
        else if (L.block_size == 32) hash_blocks_staged_kernel<32><<<n_tiles, kHashThreads, staged, stream>>>(L);
        else if (L.block_size == 64) hash_blocks_staged_kernel<64><<<n_tiles, kHashThreads, staged, stream>>>(L);
        else                         hash_blocks_staged_kernel<0><<<n_tiles, kHashThreads, staged, stream>>>(L);
    } else {
        const size_t smem = (size_t)(L.block_size + 1) * 8 +
                            (size_t)L.tile_blocks * (L.block_size / 4) * 8;
        if (vec) hash_blocks_kernel<true><<<n_tiles, kHashThreads, smem, stream>>>(L);
        else     hash_blocks_kernel<false><<<n_tiles, kHashThreads, smem, stream>>>(L);
    }
    return cudaGetLastError();
}

cudaError_t hash_kernels_init() {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (sms > 0) g_hash_sm_count = sms;
    // allow tiles whose chunk sums plus a large power table exceed the 48 KB default
    e = cudaFuncSetAttribute(hash_blocks_kernel<true>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kHashMaxSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_kernel<false>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kHashMaxSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_staged_kernel<0>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kHashStagedMaxSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_staged_kernel<16>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kHashStagedMaxSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_staged_kernel<32>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kHashStagedMaxSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_staged_kernel<64>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kHashStagedMaxSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_run_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRunSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_run_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRunSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hash_blocks_run_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRunSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(hash_blocks_tpb_kernel<false>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, kHashMaxSmem);
}

}  // namespace eakv

// ---------------------------------------------------------------------------------------
// Allocation-free block keys.
//
// Some users of this library run where device memory cannot be requested: inside a serving
// process whose engine has already claimed the GPU's memory for its KV pool (an allocation
// there can fail outright, or stall the whole device while the driver makes room), or in a
// latency-critical section that may not take the implicit synchronisation of an allocation.
// eakv_hash_blocks_static computes the same keys as eakv_hash_blocks without a context and
// without allocating anything: its scratch (block partials, the power table B^0..B^b, the
// ticket counter and a self-check word) lives in the file-scope array below, which every GPU
// that loads the library keeps resident until the process exits.
//
// The array is shared by every call on a device and keeps the previous call's contents:
// each call rewrites the power table, overwrites the partials it uses and zeroes the ticket
// counter before its kernel runs.  Two calls whose GPU work overlaps (different streams
// without an ordering between them) race on it.  The self-check word is the one thing a call
// does not clear: it stays raised until eakv_hash_blocks_static_status reads it.
// ---------------------------------------------------------------------------------------
#include "../../include/eakv.h"

#include <atomic>
#include <mutex>

namespace eakv {

constexpr int64_t kStaticMaxBlocks = EAKV_STATIC_MAX_BLOCKS;                 // 65,536 keys per call
constexpr size_t kStaticPartialBytes = (size_t)kStaticMaxBlocks * 8;          // 512 KiB
constexpr size_t kStaticPowBytes = ((size_t)(kHashMaxBlockSize + 1) * 8 + 255) / 256 * 256;
constexpr size_t kStaticCounterBytes = 256;      // ticket counter (cleared per call)
constexpr size_t kStaticFlagBytes = 256;         // self-check word (cleared only when read)
constexpr size_t kStaticBytes = kStaticPartialBytes + kStaticPowBytes + kStaticCounterBytes + kStaticFlagBytes;

// In host code this name is only a handle for cudaGetSymbolAddress, never an address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
// device address per device; published once, under g_static_mutex, after the set-up succeeded
static std::atomic<unsigned char*> g_static_ptr[kMaxDevices];
static std::mutex g_static_mutex;

// thread e writes B^e mod p
__global__ void fill_pow_table_kernel(uint64_t* pw, uint64_t base, int n_entries) {
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n_entries; e += gridDim.x * blockDim.x) {
        uint64_t r = 1, sq = base;
        for (int bits = e; bits; bits >>= 1) {
            if (bits & 1) r = mulmod61(r, sq);
            sq = mulmod61(sq, sq);
        }
        pw[e] = r;
    }
}

// The array's device address on the current device (set-up on first use), or NULL.
static unsigned char* static_scratch(int* dev_out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (dev_out) *dev_out = dev;
    unsigned char* p = g_static_ptr[dev].load(std::memory_order_acquire);
    if (p) return p;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    p = g_static_ptr[dev].load(std::memory_order_acquire);
    if (p) return p;
    // once per device, with that device current: resolve the array's device address
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || addr == nullptr) {
        cudaGetLastError();
        return nullptr;
    }
    if (hash_kernels_init() != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    g_static_ptr[dev].store(static_cast<unsigned char*>(addr), std::memory_order_release);
    return static_cast<unsigned char*>(addr);
}

}  // namespace eakv

extern "C" int eakv_hash_blocks_static(const int32_t* tokens_dev, int64_t n_tokens,
                                       int32_t block_size, uint64_t hash_base,
                                       uint64_t parent_hash, uint64_t* hashes_dev,
                                       int64_t* n_blocks_out, void* cuda_stream) {
    using namespace eakv;
    if (n_tokens < 0 || block_size <= 0 || block_size > kHashMaxBlockSize) return EAKV_E_INVAL;
    const int64_t nblk = n_tokens / block_size;
    if (n_blocks_out) *n_blocks_out = nblk;
    if (nblk > kStaticMaxBlocks) return EAKV_E_CAPACITY;   // more keys than the static scratch holds
    if (nblk == 0) return EAKV_OK;
    if (!tokens_dev || !hashes_dev) return EAKV_E_INVAL;
    if (((uintptr_t)tokens_dev & 3) || ((uintptr_t)hashes_dev & 7)) return EAKV_E_INVAL;
    if (!device_readable(tokens_dev) || !device_readable(hashes_dev)) return EAKV_E_INVAL;   // (a query, no allocation)

    unsigned char* scratch = static_scratch(nullptr);
    if (!scratch) return EAKV_E_CUDA;
    uint64_t* partial = reinterpret_cast<uint64_t*>(scratch);
    uint64_t* pw = reinterpret_cast<uint64_t*>(scratch + kStaticPartialBytes);
    int* counter = reinterpret_cast<int*>(scratch + kStaticPartialBytes + kStaticPowBytes);
    int* flag = reinterpret_cast<int*>(scratch + kStaticPartialBytes + kStaticPowBytes + kStaticCounterBytes);

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    constexpr uint64_t P = (1ull << 61) - 1;
    const uint64_t base = hash_base ? hash_base % P : 6364136223846793005ull % P;
    if (cudaMemsetAsync(counter, 0, kStaticCounterBytes, stream) != cudaSuccess) {
        cudaGetLastError();
        return EAKV_E_CUDA;
    }
    const int n_pow = block_size + 1;
    fill_pow_table_kernel<<<(n_pow + 255) / 256, 256, 0, stream>>>(pw, base, n_pow);
    if (cudaGetLastError() != cudaSuccess) return EAKV_E_CUDA;

    const bool generic = hash_thread_per_block(block_size);
    const bool vec = (block_size % 4) == 0 && (((uintptr_t)tokens_dev & 15) == 0);
    HashLaunch L;
    L.tokens = tokens_dev;
    L.keys = hashes_dev;
    L.partial = partial;
    L.counters = counter;
    L.pow_table = pw;
    L.tiles = nullptr;
    L.prompts = nullptr;
    L.single_nblk = nblk;
    L.single_parent = parent_hash % P;
    L.single_parent_ptr = nullptr;
    L.block_size = block_size;
    L.tile_blocks = hash_tile_blocks(block_size, nblk);
    L.stages = hash_stages(block_size);
    L.n_prompts = 0;
    {   // powers B^0 .. B^min(b, 64) on the host for the by-value limbs of the small-block kernels
        uint64_t pw_host[65];
        const int lim = block_size < 64 ? block_size : 64;
        pw_host[0] = 1;
        for (int e = 1; e <= lim; ++e)
            pw_host[e] = (uint64_t)(((unsigned __int128)pw_host[e - 1] * base) % P);
        if (block_size <= 64) hash_fill_limbs(L, pw_host, block_size);
        else L.pow_block = 0;   // larger blocks read B^b from the device power table
    }
    L.tokens_limit = n_tokens;
    L.blocks_limit = nblk;
    L.error_flag = flag;
    const int n_tiles = (int)((nblk + L.tile_blocks - 1) / L.tile_blocks);
    if (launch_hash(L, n_tiles, generic, vec, stream) != cudaSuccess) return EAKV_E_CUDA;
    return EAKV_OK;
}

extern "C" int eakv_hash_blocks_static_status(void* cuda_stream) {
    using namespace eakv;
    unsigned char* scratch = static_scratch(nullptr);
    if (!scratch) return EAKV_E_CUDA;
    int* flag = reinterpret_cast<int*>(scratch + kStaticPartialBytes + kStaticPowBytes + kStaticCounterBytes);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int value = 0;
    if (cudaMemcpyAsync(&value, flag, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return EAKV_E_CUDA;
    }
    if (value == 0) return EAKV_OK;
    if (cudaMemsetAsync(flag, 0, sizeof(int), stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return EAKV_E_CUDA;
    }
    return EAKV_E_RANGE;
}
