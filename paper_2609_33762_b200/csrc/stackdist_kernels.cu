// Stack-distance capacity model on the GPU (Section 3.2, Eq. 4; Appendix C "Prefix coverage
// from a reference stream").
//
// Reuse distance of reference i with previous reference p to the same chunk: how many different
// chunks, other than this one, are touched strictly between the two.  A position j in (p, i) is the
// first reference to its chunk inside that window exactly when its own previous reference lies
// before p, and every j <= p trivially has prev_j < p, so
//
//     D_i = #{ j < i : prev_j < p } - (p + 1).
//
// Steps, all data-parallel:
//   1. prev[]: stable sort of (key, position) pairs by key (a least-significant-digit radix sort
//      written here: eight passes of 8 bits, three kernels per pass, no kernel waits for another);
//      equal neighbours give each position its predecessor.
//   2. a wavelet matrix over v_j = prev_j + 1 (one stable 0/1 partition per bit, built with a
//      three-kernel exclusive scan per level: no kernel waits for another);
//   3. one "count of values below x in a prefix" query per reference, nbits steps each.
// The capacity curve then needs only D: a reference hits a tier of K chunks iff D < K
// (Mattson); the host-covered prefix of a request = its leading run of hits; restored = max(0, H - G);
// computed prefill = n - max(G, H) * b.
#include <algorithm>
#include <climits>
#include <cstdint>
#include <vector>

#include "../../include/eakv.h"
#include "eakv_internal.h"

namespace eakv {

constexpr int kSdThreads = 256;
constexpr int kSdItems = 4;                         // elements per thread in the scan kernels
constexpr int kSdTile = kSdThreads * kSdItems;      // 1024 elements per CTA

// ---- step 1: stable LSD radix sort of (key, position) ---------------------------------------
// One pass sorts by the 8-bit digit at `shift`.  A CTA owns a tile of kRsTile consecutive
// elements.  (a) per-tile digit counts, stored digit-major: counts[digit][tile]; (b) one CTA per
// digit turns its row into exclusive offsets across tiles and leaves the digit's total; (c) every
// CTA scans the 256 totals into digit bases, then walks its tile in rounds of kRsThreads elements
// in order, ranking equal digits by (round, warp, lane) so that the pass is stable, and scatters.
constexpr int kRsThreads = 256;
constexpr int kRsItems = 8;
constexpr int kRsTile = kRsThreads * kRsItems;      // 2048 elements per CTA
constexpr int kRsDigits = 256;

__global__ void __launch_bounds__(kRsThreads)
rs_count_kernel(const uint64_t* __restrict__ keys, int64_t n, int shift, int n_tiles,
                int32_t* __restrict__ counts /* [256][n_tiles] */) {
    __shared__ int hist[kRsDigits];
    hist[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kRsTile;
#pragma unroll
    for (int k = 0; k < kRsItems; ++k) {
        const int64_t i = base + k * kRsThreads + threadIdx.x;
        if (i < n) atomicAdd(&hist[(int)((keys[i] >> shift) & 255u)], 1);
    }
    __syncthreads();
    counts[(int64_t)threadIdx.x * n_tiles + blockIdx.x] = hist[threadIdx.x];
}

// one CTA per digit: exclusive scan of its row of tile counts (in place), total to totals[digit]
__global__ void __launch_bounds__(1024)
rs_scan_rows_kernel(int32_t* __restrict__ counts, int n_tiles, int32_t* __restrict__ totals) {
    __shared__ int warp_tot[32];
    __shared__ int carry_s;
    int32_t* row = counts + (int64_t)blockIdx.x * n_tiles;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < n_tiles; base += 1024) {
        const int i = base + threadIdx.x;
        const int x = i < n_tiles ? row[i] : 0;
        int inc = x;
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += up;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            int w = warp_tot[lane];
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, w, d);
                if (lane >= d) w += up;
            }
            warp_tot[lane] = w;
        }
        __syncthreads();
        const int carry = carry_s;
        if (i < n_tiles) row[i] = carry + (warp ? warp_tot[warp - 1] : 0) + inc - x;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = carry + warp_tot[31];
        __syncthreads();
    }
    if (threadIdx.x == 0) totals[blockIdx.x] = carry_s;
}

// idx_in == NULL: the value of element i is its position i (first pass)
__global__ void __launch_bounds__(kRsThreads)
rs_scatter_kernel(const uint64_t* __restrict__ keys_in, const int32_t* __restrict__ idx_in, int64_t n,
                  int shift, int n_tiles, const int32_t* __restrict__ counts /* exclusive, [256][n_tiles] */,
                  const int32_t* __restrict__ totals, uint64_t* __restrict__ keys_out,
                  int32_t* __restrict__ idx_out) {
    __shared__ int digit_base[kRsDigits];            // where this tile's elements of a digit start
    __shared__ int warp_count[kRsThreads / 32][kRsDigits];
    __shared__ int scan_tmp[kRsThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    {   // exclusive scan of the 256 digit totals + this tile's offset inside each digit
        const int t = totals[tid];
        int inc = t;
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += up;
        }
        if (lane == 31) scan_tmp[warp] = inc;
        __syncthreads();
        int before = inc - t;
        for (int w = 0; w < warp; ++w) before += scan_tmp[w];
        digit_base[tid] = before + counts[(int64_t)tid * n_tiles + blockIdx.x];
    }
    for (int w = 0; w < kRsThreads / 32; ++w) warp_count[w][tid] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kRsTile;
    for (int k = 0; k < kRsItems; ++k) {
        const int64_t i = base + k * kRsThreads + tid;
        const bool live = i < n;
        const uint64_t key = live ? keys_in[i] : 0;
        const int d = live ? (int)((key >> shift) & 255u) : -1;
        // lanes of this warp with the same digit; dead lanes (d = -1) only match each other
        const unsigned peers = __match_any_sync(0xffffffffu, d);
        const int rank = __popc(peers & ((1u << lane) - 1u));
        if (live && rank == 0) warp_count[warp][d] = __popc(peers);
        __syncthreads();
        if (live) {
            int off = digit_base[d] + rank;
            for (int w = 0; w < warp; ++w) off += warp_count[w][d];
            keys_out[off] = key;
            idx_out[off] = idx_in ? idx_in[i] : (int32_t)i;
        }
        __syncthreads();
        {   // this round's elements of digit `tid` are placed: advance the base, clear the counts
            int sum = 0;
            for (int w = 0; w < kRsThreads / 32; ++w) {
                sum += warp_count[w][tid];
                warp_count[w][tid] = 0;
            }
            digit_base[tid] += sum;
        }
        __syncthreads();
    }
}

// sorted by (key, position): the predecessor of a position is its left neighbour with the same key
// (and its successor, when asked for, the right neighbour with the same key)
__global__ void prev_from_sorted_kernel(const uint64_t* __restrict__ keys_sorted,
                                        const int32_t* __restrict__ idx_sorted, int64_t n,
                                        int32_t* __restrict__ prev, uint32_t* __restrict__ v,
                                        int32_t* __restrict__ next /* or NULL */) {
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n) return;
    const int32_t i = idx_sorted[s];
    const int32_t p = (s > 0 && keys_sorted[s - 1] == keys_sorted[s]) ? idx_sorted[s - 1] : -1;
    prev[i] = p;
    v[i] = (uint32_t)(p + 1);
    if (next) next[i] = (s + 1 < n && keys_sorted[s + 1] == keys_sorted[s]) ? idx_sorted[s + 1] : -1;
}

// Declined-chunk audit (Appendix D, "Reuse distance of declined chunks"): for every declined
// position, the reuse distance at which its chunk is referenced next.  counts[0] = declined
// positions, counts[1] = those whose next reference lies at D >= capacity or never comes (the
// condition of Proposition 1), counts[2] = those never referenced again.
__global__ void declined_audit_kernel(const uint8_t* __restrict__ declined, const int32_t* __restrict__ next,
                                      const int64_t* __restrict__ dist, int64_t n, int64_t capacity,
                                      int64_t* __restrict__ next_dist /* or NULL */,
                                      unsigned long long* __restrict__ counts) {
    unsigned long long c0 = 0, c1 = 0, c2 = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (int64_t)gridDim.x * blockDim.x) {
        int64_t out = -2;                       // not declined
        if (declined[i]) {
            const int32_t j = next[i];
            ++c0;
            if (j < 0) {
                ++c1; ++c2;
                out = -1;                       // never referenced again
            } else {
                out = dist[j];
                if (out >= capacity) ++c1;
            }
        }
        if (next_dist) next_dist[i] = out;
    }
    for (int d = 16; d; d >>= 1) {
        c0 += __shfl_xor_sync(0xffffffffu, c0, d);
        c1 += __shfl_xor_sync(0xffffffffu, c1, d);
        c2 += __shfl_xor_sync(0xffffffffu, c2, d);
    }
    if ((threadIdx.x & 31) == 0) {
        if (c0) atomicAdd(&counts[0], c0);
        if (c1) atomicAdd(&counts[1], c1);
        if (c2) atomicAdd(&counts[2], c2);
    }
}

// ---- step 2: one wavelet-matrix level = stable partition by one bit -------------------------
// pass A: zeros per tile
__global__ void __launch_bounds__(kSdThreads)
wm_count_kernel(const uint32_t* __restrict__ a, int64_t n, int shift, int32_t* __restrict__ tile_zeros) {
    __shared__ int warp_sum[kSdThreads / 32];
    const int64_t base = (int64_t)blockIdx.x * kSdTile;
    int z = 0;
#pragma unroll
    for (int k = 0; k < kSdItems; ++k) {
        const int64_t i = base + (int64_t)threadIdx.x * kSdItems + k;
        if (i < n) z += ((a[i] >> shift) & 1u) ^ 1u;
    }
    for (int d = 16; d; d >>= 1) z += __shfl_xor_sync(0xffffffffu, z, d);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = z;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < kSdThreads / 32; ++w) t += warp_sum[w];
        tile_zeros[blockIdx.x] = t;
    }
}

// pass B: exclusive scan of the tile counts by one CTA (in place), total to *total_zeros
__global__ void __launch_bounds__(1024)
wm_scan_tiles_kernel(int32_t* __restrict__ tile_zeros, int n_tiles, int32_t* __restrict__ total_zeros) {
    __shared__ int warp_tot[32];
    __shared__ int carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < n_tiles; base += 1024) {
        const int i = base + threadIdx.x;
        const int x = i < n_tiles ? tile_zeros[i] : 0;
        int inc = x;
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += up;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            int w = warp_tot[lane];
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, w, d);
                if (lane >= d) w += up;
            }
            warp_tot[lane] = w;
        }
        __syncthreads();
        const int carry = carry_s;
        const int excl = carry + (warp ? warp_tot[warp - 1] : 0) + inc - x;
        if (i < n_tiles) tile_zeros[i] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = carry + warp_tot[31];
        __syncthreads();
    }
    if (threadIdx.x == 0) *total_zeros = carry_s;
}

// pass C: zeros-before for every position, and the scatter into the next level's order
__global__ void __launch_bounds__(kSdThreads)
wm_scatter_kernel(const uint32_t* __restrict__ a, int64_t n, int shift,
                  const int32_t* __restrict__ tile_excl, const int32_t* __restrict__ total_zeros,
                  int32_t* __restrict__ zeros_before /* [n + 1] */, uint32_t* __restrict__ a_next) {
    __shared__ int warp_tot[kSdThreads / 32];
    const int64_t base = (int64_t)blockIdx.x * kSdTile + (int64_t)threadIdx.x * kSdItems;
    uint32_t val[kSdItems];
    int isz[kSdItems];
    int mine = 0;
#pragma unroll
    for (int k = 0; k < kSdItems; ++k) {
        const int64_t i = base + k;
        val[k] = i < n ? a[i] : 0xffffffffu;
        isz[k] = (i < n) ? (int)(((val[k] >> shift) & 1u) ^ 1u) : 0;
        mine += isz[k];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = mine;
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += up;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    int before = tile_excl[blockIdx.x] + inc - mine;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    const int z_total = *total_zeros;
#pragma unroll
    for (int k = 0; k < kSdItems; ++k) {
        const int64_t i = base + k;
        if (i < n) {
            zeros_before[i] = before;
            const int64_t dst = isz[k] ? (int64_t)before : (int64_t)z_total + (i - before);
            a_next[dst] = val[k];
            before += isz[k];
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) zeros_before[n] = z_total;   // zeros in the whole level
}

// ---- step 3 ---------------------------------------------------------------------------------
// dist[i] = #{ j < i : v_j < p + 1 } - (p + 1), or -1 on a first reference
__global__ void reuse_distance_kernel(const int32_t* __restrict__ prev, int64_t n, int nbits,
                                      const int32_t* __restrict__ zeros_before /* [nbits][n+1] */,
                                      const int32_t* __restrict__ level_zeros /* [nbits] */,
                                      int64_t* __restrict__ dist) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t p = prev[i];
    if (p < 0) {
        dist[i] = -1;
        return;
    }
    const uint32_t x = (uint32_t)p + 1u;
    int64_t lo = 0, hi = i, count = 0;
    for (int l = 0; l < nbits; ++l) {
        const int32_t* zb = zeros_before + (int64_t)l * (n + 1);
        const int64_t z_lo = zb[lo], z_hi = zb[hi];
        if ((x >> (nbits - 1 - l)) & 1u) {
            count += z_hi - z_lo;
            const int64_t z = level_zeros[l];
            lo = z + (lo - z_lo);
            hi = z + (hi - z_hi);
        } else {
            lo = z_lo;
            hi = z_hi;
        }
    }
    dist[i] = count - ((int64_t)p + 1);
}

// largest finite reuse distance of the stream (-1 if every reference is a first reference)
__global__ void max_distance_kernel(const int64_t* __restrict__ dist, int64_t n, long long* __restrict__ out) {
    long long m = -1;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        m = max(m, (long long)dist[i]);
    for (int d = 16; d; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
    if ((threadIdx.x & 31) == 0 && m >= 0) atomicMax(out, m);
}

// ---- capacity curve ---------------------------------------------------------------------------
// hits[c] += #{ i : 0 <= D_i < K_c }
__global__ void curve_hits_kernel(const int64_t* __restrict__ dist, int64_t n,
                                  const int64_t* __restrict__ caps, int n_caps,
                                  unsigned long long* __restrict__ hits) {
    extern __shared__ unsigned long long sh[];
    for (int c = threadIdx.x; c < n_caps; c += blockDim.x) sh[c] = 0;
    __syncthreads();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t d = dist[i];
        if (d < 0) continue;
        for (int c = 0; c < n_caps; ++c)
            if (d < caps[c]) atomicAdd(&sh[c], 1ull);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < n_caps; c += blockDim.x)
        if (sh[c]) atomicAdd(&hits[c], sh[c]);
}

// one CTA per request: running maximum of D over the request's references (a first reference
// counts as infinite), coverage H(K) = references before the maximum reaches K
__global__ void __launch_bounds__(kSdThreads)
curve_cover_kernel(const int64_t* __restrict__ dist, const int64_t* __restrict__ req_off,
                   const int64_t* __restrict__ req_tokens, const int64_t* __restrict__ req_gpu,
                   int64_t n_req, int block_size, const int64_t* __restrict__ caps, int n_caps,
                   unsigned long long* __restrict__ restored, unsigned long long* __restrict__ computed,
                   int64_t* __restrict__ cover /* [n_caps][n_req] or NULL */) {
    __shared__ long long warp_max[kSdThreads / 32];
    __shared__ long long carry_s;
    __shared__ int cnt[64];
    const int64_t r = blockIdx.x;
    if (r >= n_req) return;
    const int64_t lo = req_off[r], hi = req_off[r + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = -1;
    for (int c = threadIdx.x; c < n_caps; c += blockDim.x) cnt[c] = 0;
    __syncthreads();
    const long long INF = 0x7fffffffffffffffLL;
    for (int64_t base = lo; base < hi; base += kSdThreads) {
        const int64_t i = base + threadIdx.x;
        long long m = -1;
        if (i < hi) {
            const long long d = dist[i];
            m = d < 0 ? INF : d;
        }
        for (int d = 1; d < 32; d <<= 1) {
            const long long up = __shfl_up_sync(0xffffffffu, m, d);
            if (lane >= d) m = max(m, up);
        }
        if (lane == 31) warp_max[warp] = m;
        __syncthreads();
        long long pm = max(m, carry_s);
        for (int w = 0; w < warp; ++w) pm = max(pm, warp_max[w]);
        if (i < hi) {
            for (int c = 0; c < n_caps; ++c)
                if (pm < caps[c]) atomicAdd(&cnt[c], 1);
        }
        __syncthreads();
        if (threadIdx.x == kSdThreads - 1) carry_s = pm;
        __syncthreads();
    }
    if (threadIdx.x < n_caps) {
        const int c = threadIdx.x;
        const long long H = cnt[c], G = req_gpu[r], n = req_tokens[r];
        if (cover) cover[(int64_t)c * n_req + r] = H;
        if (H > G) atomicAdd(&restored[c], (unsigned long long)(H - G));
        atomicAdd(&computed[c], (unsigned long long)(n - max(G, H) * (long long)block_size));
    }
}

}  // namespace eakv

using namespace eakv;

#define SD_CU(call)                           \
    do {                                      \
        cudaError_t _e = (call);              \
        if (_e != cudaSuccess) {              \
            rc = EAKV_E_CUDA;                 \
            goto done;                        \
        }                                     \
    } while (0)

// dist_dev[i] for all references; next_dev (optional, int32[n]) receives the position of the next
// reference to the same key or -1.  Returns after the stream has finished the work.
static int reuse_distances_impl(const uint64_t* keys_dev, int64_t n_refs, int64_t* dist_dev,
                                int32_t* next_dev, cudaStream_t stream) {
    const int64_t n = n_refs;
    int nbits = 1;
    while ((1ll << nbits) <= n) ++nbits;               // values v in [0, n] fit in nbits bits
    const int n_tiles = (int)((n + kSdTile - 1) / kSdTile);
    const int grid1 = (int)((n + 255) / 256);

    int rc = EAKV_OK;
    uint64_t *keys_sorted = nullptr, *keys_tmp = nullptr;
    int32_t *idx_tmp = nullptr, *idx_sorted = nullptr, *prev = nullptr, *zeros_before = nullptr;
    int32_t *tile_zeros = nullptr, *level_zeros = nullptr, *rs_counts = nullptr, *rs_totals = nullptr;
    uint32_t *va = nullptr, *vb = nullptr;
    const int rs_tiles = (int)((n + kRsTile - 1) / kRsTile);

    SD_CU(cudaMalloc(&keys_sorted, n * 8));
    SD_CU(cudaMalloc(&keys_tmp, n * 8));
    SD_CU(cudaMalloc(&idx_tmp, n * 4));
    SD_CU(cudaMalloc(&idx_sorted, n * 4));
    SD_CU(cudaMalloc(&prev, n * 4));
    SD_CU(cudaMalloc(&va, n * 4));
    SD_CU(cudaMalloc(&vb, n * 4));
    SD_CU(cudaMalloc(&zeros_before, (size_t)nbits * (n + 1) * 4));
    SD_CU(cudaMalloc(&tile_zeros, (size_t)n_tiles * 4));
    SD_CU(cudaMalloc(&level_zeros, (size_t)nbits * 4));
    SD_CU(cudaMalloc(&rs_counts, (size_t)kRsDigits * rs_tiles * 4));
    SD_CU(cudaMalloc(&rs_totals, kRsDigits * 4));

    // eight stable passes over the 61-bit keys, least significant digit first; the buffers alternate
    // so that the last pass lands in keys_sorted / idx_sorted
    for (int pass = 0; pass < 8; ++pass) {
        const uint64_t* kin = pass == 0 ? keys_dev : ((pass & 1) ? keys_tmp : keys_sorted);
        const int32_t* iin = pass == 0 ? nullptr : ((pass & 1) ? idx_tmp : idx_sorted);
        uint64_t* kout = (pass & 1) ? keys_sorted : keys_tmp;
        int32_t* iout = (pass & 1) ? idx_sorted : idx_tmp;
        rs_count_kernel<<<rs_tiles, kRsThreads, 0, stream>>>(kin, n, 8 * pass, rs_tiles, rs_counts);
        rs_scan_rows_kernel<<<kRsDigits, 1024, 0, stream>>>(rs_counts, rs_tiles, rs_totals);
        rs_scatter_kernel<<<rs_tiles, kRsThreads, 0, stream>>>(kin, iin, n, 8 * pass, rs_tiles, rs_counts, rs_totals,
                                                               kout, iout);
    }
    prev_from_sorted_kernel<<<grid1, 256, 0, stream>>>(keys_sorted, idx_sorted, n, prev, va, next_dev);
    for (int l = 0; l < nbits; ++l) {
        const int shift = nbits - 1 - l;
        uint32_t* a = (l & 1) ? vb : va;
        uint32_t* a_next = (l & 1) ? va : vb;
        wm_count_kernel<<<n_tiles, kSdThreads, 0, stream>>>(a, n, shift, tile_zeros);
        wm_scan_tiles_kernel<<<1, 1024, 0, stream>>>(tile_zeros, n_tiles, level_zeros + l);
        wm_scatter_kernel<<<n_tiles, kSdThreads, 0, stream>>>(a, n, shift, tile_zeros, level_zeros + l,
                                                             zeros_before + (int64_t)l * (n + 1), a_next);
    }
    reuse_distance_kernel<<<grid1, 256, 0, stream>>>(prev, n, nbits, zeros_before, level_zeros, dist_dev);
    SD_CU(cudaGetLastError());
    SD_CU(cudaStreamSynchronize(stream));
done:
    cudaFree(keys_sorted); cudaFree(keys_tmp); cudaFree(idx_tmp); cudaFree(idx_sorted); cudaFree(prev);
    cudaFree(va); cudaFree(vb); cudaFree(zeros_before); cudaFree(tile_zeros); cudaFree(level_zeros);
    cudaFree(rs_counts); cudaFree(rs_totals);
    if (rc != EAKV_OK) cudaGetLastError();
    return rc;
}

extern "C" int eakv_reuse_distances(const uint64_t* keys_dev, int64_t n_refs, int64_t* dist_dev,
                                    void* cuda_stream) {
    if (n_refs < 0 || n_refs > 0x7ffffff0LL) return EAKV_E_INVAL;
    if (n_refs == 0) return EAKV_OK;
    if (!keys_dev || !dist_dev) return EAKV_E_INVAL;
    if (!device_readable(keys_dev) || !device_readable(dist_dev)) return EAKV_E_INVAL;
    return reuse_distances_impl(keys_dev, n_refs, dist_dev, nullptr, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int eakv_declined_audit(const uint64_t* keys_dev, const uint8_t* declined_dev, int64_t n_refs,
                                   int64_t capacity, int64_t* declined_out, int64_t* meets_out,
                                   int64_t* never_out, int64_t* next_dist_dev, void* cuda_stream) {
    if (n_refs < 0 || n_refs > 0x7ffffff0LL || capacity < 0) return EAKV_E_INVAL;
    if (!declined_out || !meets_out || !never_out) return EAKV_E_INVAL;
    *declined_out = *meets_out = *never_out = 0;
    if (n_refs == 0) return EAKV_OK;
    if (!keys_dev || !declined_dev) return EAKV_E_INVAL;
    if (!device_readable(keys_dev) || !device_readable(declined_dev) ||
        (next_dist_dev && !device_readable(next_dist_dev)))
        return EAKV_E_INVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = EAKV_OK;
    int64_t* dist = nullptr;
    int32_t* next = nullptr;
    unsigned long long* counts = nullptr;
    unsigned long long host_counts[3] = {0, 0, 0};
    int dev = 0, sms = 148;
    SD_CU(cudaMalloc(&dist, n_refs * 8));
    SD_CU(cudaMalloc(&next, n_refs * 4));
    SD_CU(cudaMalloc(&counts, 3 * 8));
    SD_CU(cudaMemsetAsync(counts, 0, 3 * 8, stream));
    rc = reuse_distances_impl(keys_dev, n_refs, dist, next, stream);
    if (rc != EAKV_OK) goto done;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    declined_audit_kernel<<<(int)std::min<int64_t>((n_refs + 255) / 256, (int64_t)sms * 8), 256, 0, stream>>>(
        declined_dev, next, dist, n_refs, capacity, next_dist_dev, counts);
    SD_CU(cudaGetLastError());
    SD_CU(cudaMemcpyAsync(host_counts, counts, 3 * 8, cudaMemcpyDeviceToHost, stream));
    SD_CU(cudaStreamSynchronize(stream));
    *declined_out = (int64_t)host_counts[0];
    *meets_out = (int64_t)host_counts[1];
    *never_out = (int64_t)host_counts[2];
done:
    cudaFree(dist); cudaFree(next); cudaFree(counts);
    if (rc != EAKV_OK) cudaGetLastError();
    return rc;
}

extern "C" int eakv_working_set(const eakv_working_set_in* in, eakv_working_set_out* out) {
    if (!in || !out) return EAKV_E_INVAL;
    if (in->num_layers <= 0 || in->kv_heads <= 0 || in->head_dim <= 0 || in->elem_bytes <= 0 ||
        in->tensor_parallel <= 0 || in->block_size <= 0 || in->active_pool <= 0 || in->n_requests <= 0 ||
        in->total_prompt_tokens < 0 || in->gpu_blocks < 0 || in->host_blocks < 0)
        return EAKV_E_INVAL;
    typedef __int128 wide;
    // Eq. 1: beta_rank = 2 L d s max(1, ceil(H_kv / TP))
    const int64_t heads = std::max<int64_t>(1, (in->kv_heads + in->tensor_parallel - 1) / in->tensor_parallel);
    const int64_t beta = 2ll * in->num_layers * in->head_dim * in->elem_bytes * heads;
    // Eq. 5 with N_bar = total / requests kept as a fraction: (A - 1) * total * beta / requests
    const wide num = (wide)(in->active_pool - 1) * in->total_prompt_tokens;
    out->beta_rank_bytes = beta;
    out->working_set_bytes = (int64_t)(num * beta / in->n_requests);
    out->working_set_blocks = (int64_t)(num / ((wide)in->n_requests * in->block_size));
    // gamma_G = A * N_bar / K_G with K_G = gpu_blocks * b tokens; gamma_H = C_reuse / C_H with
    // C_H = host_blocks * b * beta (beta cancels)
    const wide g_num = (wide)in->active_pool * in->total_prompt_tokens;
    const wide g_den = (wide)in->n_requests * in->gpu_blocks * in->block_size;
    const wide h_den = (wide)in->n_requests * in->host_blocks * in->block_size;
    out->gamma_g = g_den ? (double)g_num / (double)g_den : 0.0;
    out->gamma_h = h_den ? (double)num / (double)h_den : 0.0;
    out->pool_exceeds_gpu = g_den ? (g_num > g_den) : 0;
    out->working_set_exceeds_host = h_den ? (num > h_den) : 0;
    return EAKV_OK;
}

extern "C" int eakv_offload_benefit(const eakv_offload_in* in, eakv_offload_out* out) {
    if (!in || !out) return EAKV_E_INVAL;
    if (in->prefix_tokens <= 0 || in->beta_rank_bytes <= 0 || in->t_prefill_ps <= 0 ||
        in->h2d_bytes_per_s <= 0 || in->tau_load_ps < 0)
        return EAKV_E_INVAL;
    typedef __int128 wide;
    const wide ps = 1000000000000ll;
    // Eq. 2: T_load(n) = n * beta / B_H2D + tau_load,  T_rec(n) = n * t_pf  (picoseconds, floor)
    const wide load = (wide)in->prefix_tokens * in->beta_rank_bytes * ps / in->h2d_bytes_per_s + in->tau_load_ps;
    const wide rec = (wide)in->prefix_tokens * in->t_prefill_ps;
    const wide lim = (wide)INT64_MAX;
    out->t_load_ps = (int64_t)std::min(load, lim);
    out->t_rec_ps = (int64_t)std::min(rec, lim);
    out->obr = 1.0 - (double)load / (double)rec;
    out->restore_is_faster = load < rec;
    // per token: beta / B_H2D against t_pf, compared as beta * 10^12 against t_pf * B_H2D; the fixed
    // cost tau is repaid after n* = ceil(tau * B_H2D / (t_pf * B_H2D - beta * 10^12)) tokens
    const wide load_b = (wide)in->beta_rank_bytes * ps;
    const wide rec_b = (wide)in->t_prefill_ps * in->h2d_bytes_per_s;
    out->obr_long_prefix = 1.0 - (double)load_b / (double)rec_b;
    if (load_b >= rec_b) {
        out->break_even_tokens = -1;                 // a restored token never costs less than a computed one
    } else {
        const wide gain = rec_b - load_b;
        out->break_even_tokens = (int64_t)std::min(((wide)in->tau_load_ps * in->h2d_bytes_per_s + gain - 1) / gain, lim);
    }
    return EAKV_OK;
}

extern "C" int eakv_capacity_curve(const int64_t* dist_dev, int64_t n_refs,
                                   const int64_t* req_offsets_host, const int64_t* req_tokens_host,
                                   const int64_t* req_gpu_prefix_host, int64_t n_requests,
                                   int32_t block_size, const int64_t* capacities_host,
                                   int32_t n_capacities, int64_t* hits_out, int64_t* restored_out,
                                   int64_t* computed_out, int64_t* cover_out, void* cuda_stream) {
    if (n_refs < 0 || n_requests < 0 || n_capacities <= 0 || n_capacities > 64 || block_size <= 0)
        return EAKV_E_INVAL;
    if (!req_offsets_host || !capacities_host || !hits_out || !restored_out || !computed_out)
        return EAKV_E_INVAL;
    if (n_requests > 0 && (!req_tokens_host || !req_gpu_prefix_host)) return EAKV_E_INVAL;
    if (n_refs > 0 && !dist_dev) return EAKV_E_INVAL;
    if (n_refs > 0 && !device_readable(dist_dev)) return EAKV_E_INVAL;
    if (req_offsets_host[0] != 0 || req_offsets_host[n_requests] != n_refs) return EAKV_E_INVAL;
    for (int64_t r = 0; r < n_requests; ++r)
        if (req_offsets_host[r + 1] < req_offsets_host[r]) return EAKV_E_INVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = EAKV_OK;
    int64_t *d_off = nullptr, *d_tok = nullptr, *d_gpu = nullptr, *d_caps = nullptr, *d_cover = nullptr;
    unsigned long long* d_out = nullptr;     // hits | restored | computed
    std::vector<unsigned long long> out(3 * (size_t)n_capacities);
    const int C = n_capacities;

    SD_CU(cudaMalloc(&d_off, (n_requests + 1) * 8));
    SD_CU(cudaMalloc(&d_tok, std::max<int64_t>(n_requests, 1) * 8));
    SD_CU(cudaMalloc(&d_gpu, std::max<int64_t>(n_requests, 1) * 8));
    SD_CU(cudaMalloc(&d_caps, C * 8));
    SD_CU(cudaMalloc(&d_out, 3 * C * 8));
    if (cover_out) SD_CU(cudaMalloc(&d_cover, std::max<int64_t>((int64_t)C * n_requests, 1) * 8));
    SD_CU(cudaMemcpyAsync(d_off, req_offsets_host, (n_requests + 1) * 8, cudaMemcpyHostToDevice, stream));
    if (n_requests) {
        SD_CU(cudaMemcpyAsync(d_tok, req_tokens_host, n_requests * 8, cudaMemcpyHostToDevice, stream));
        SD_CU(cudaMemcpyAsync(d_gpu, req_gpu_prefix_host, n_requests * 8, cudaMemcpyHostToDevice, stream));
    }
    SD_CU(cudaMemcpyAsync(d_caps, capacities_host, C * 8, cudaMemcpyHostToDevice, stream));
    SD_CU(cudaMemsetAsync(d_out, 0, 3 * C * 8, stream));
    if (n_refs > 0) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int grid = (int)std::min<int64_t>((n_refs + 255) / 256, (int64_t)sms * 8);
        curve_hits_kernel<<<grid, 256, C * 8, stream>>>(dist_dev, n_refs, d_caps, C, d_out);
    }
    if (n_requests > 0) {
        curve_cover_kernel<<<(unsigned)n_requests, kSdThreads, 0, stream>>>(
            dist_dev, d_off, d_tok, d_gpu, n_requests, block_size, d_caps, C, d_out + C, d_out + 2 * C,
            d_cover);
    }
    SD_CU(cudaGetLastError());
    SD_CU(cudaMemcpyAsync(out.data(), d_out, 3 * C * 8, cudaMemcpyDeviceToHost, stream));
    if (cover_out && n_requests)
        SD_CU(cudaMemcpyAsync(cover_out, d_cover, (size_t)C * n_requests * 8, cudaMemcpyDeviceToHost, stream));
    SD_CU(cudaStreamSynchronize(stream));
    for (int c = 0; c < C; ++c) {
        hits_out[c] = (int64_t)out[c];
        restored_out[c] = (int64_t)out[C + c];
        computed_out[c] = (int64_t)out[2 * C + c];
    }
done:
    cudaFree(d_off); cudaFree(d_tok); cudaFree(d_gpu); cudaFree(d_caps); cudaFree(d_out); cudaFree(d_cover);
    if (rc != EAKV_OK) cudaGetLastError();
    return rc;
}

// Working-set sizes read off the distances (Section 3.2: the capacity at which more host memory
// stops paying).  full = largest finite reuse distance + 1, the smallest tier that hits every
// re-reference.  within = the smallest tier whose predicted computed prefill is within `percent`
// per cent of the unbounded tier's: computed prefill never grows with capacity, so the condition is
// monotone and the bracket (fails, passes] is narrowed with 64 capacities per curve launch.
extern "C" int eakv_working_set_sizes(const int64_t* dist_dev, int64_t n_refs, const int64_t* req_offsets_host,
                                      const int64_t* req_tokens_host, const int64_t* req_gpu_prefix_host,
                                      int64_t n_requests, int32_t block_size, int32_t percent,
                                      int64_t* full_out, int64_t* within_out, void* cuda_stream) {
    if (n_refs < 0 || n_requests < 0 || block_size <= 0 || percent < 0 || !full_out || !within_out)
        return EAKV_E_INVAL;
    if (n_refs > 0 && !dist_dev) return EAKV_E_INVAL;
    if (n_refs > 0 && !device_readable(dist_dev)) return EAKV_E_INVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = EAKV_OK;
    long long* d_max = nullptr;
    long long h_max = -1;
    int dev = 0, sms = 148;
    SD_CU(cudaMalloc(&d_max, 8));
    SD_CU(cudaMemcpyAsync(d_max, &h_max, 8, cudaMemcpyHostToDevice, stream));
    if (n_refs > 0) {
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        max_distance_kernel<<<(int)std::min<int64_t>((n_refs + 255) / 256, (int64_t)sms * 8), 256, 0, stream>>>(
            dist_dev, n_refs, d_max);
        SD_CU(cudaGetLastError());
    }
    SD_CU(cudaMemcpyAsync(&h_max, d_max, 8, cudaMemcpyDeviceToHost, stream));
    SD_CU(cudaStreamSynchronize(stream));
done:
    cudaFree(d_max);
    if (rc != EAKV_OK) {
        cudaGetLastError();
        return rc;
    }
    const int64_t full = h_max + 1;
    *full_out = full;
    auto computed_at = [&](const std::vector<int64_t>& caps, std::vector<int64_t>& out) -> int {
        std::vector<int64_t> hits(caps.size()), restored(caps.size());
        out.resize(caps.size());
        return eakv_capacity_curve(dist_dev, n_refs, req_offsets_host, req_tokens_host, req_gpu_prefix_host,
                                   n_requests, block_size, caps.data(), (int32_t)caps.size(), hits.data(),
                                   restored.data(), out.data(), nullptr, cuda_stream);
    };
    std::vector<int64_t> caps{std::max<int64_t>(full, 1)}, computed;
    rc = computed_at(caps, computed);
    if (rc != EAKV_OK) return rc;
    const __int128 floor_tokens = computed[0];
    auto passes = [&](int64_t c) { return (__int128)c * 100 <= floor_tokens * (100 + percent); };
    int64_t lo = -1, hi = std::max<int64_t>(full, 0);              // lo fails (or is below 0), hi passes
    while (hi - lo > 1) {
        const int64_t span = hi - lo;
        caps.clear();
        for (int i = 1; i <= 64; ++i) {
            const int64_t c = lo + std::max<int64_t>(1, (int64_t)((__int128)span * i / 65));
            if (c < hi && (caps.empty() || c > caps.back())) caps.push_back(c);
        }
        if (caps.empty()) break;
        std::vector<int64_t> query(caps);
        for (int64_t& c : query) c = std::max<int64_t>(c, 0);
        rc = computed_at(query, computed);
        if (rc != EAKV_OK) return rc;
        for (size_t i = 0; i < caps.size(); ++i) {
            if (passes(computed[i])) { hi = caps[i]; break; }      // the first that passes bounds from above
            lo = caps[i];                                          // everything before it fails
        }
    }
    *within_out = hi;
    return EAKV_OK;
}
