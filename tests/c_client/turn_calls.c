/* The two-call turn engine from plain C: eakv_turn_begin / eakv_turn_end on a tiny KV shape.
 *
 * Turn 1: a prompt of 6 full blocks + 4 tokens; the "engine" fills every block flagged needs_fill
 *         with a pattern derived from the block's key, the turn ends (host write).
 * Turn 2: another prompt that takes turn 1's blocks off the 8-block GPU tier.
 * Turn 3: turn 1's prompt again, grown by one block: its first 6 blocks come back from the host
 *         tier (restore inside eakv_turn_begin), only the new block is flagged for the engine.
 * Prints the view's scalars per turn and whether the restored GPU blocks hold the pattern of
 * their keys.  Exit code 0 when every call returned EAKV_OK and the bytes are right.
 */
#include <cuda_runtime_api.h>
#include <inttypes.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "eakv.h"

enum { L = 2, HEADS = 1, DIM = 32, B = 16, ELEM = 2, NB = 8, KH = 32 };
#define PIECE ((size_t)B * HEADS * DIM * ELEM)

#define CK(call)                                                                            \
    do {                                                                                    \
        int rc_ = (call);                                                                   \
        if (rc_ != EAKV_OK) {                                                               \
            fprintf(stderr, "%s -> %d (%s)\n", #call, rc_, eakv_strerror(rc_));             \
            return 2;                                                                       \
        }                                                                                   \
    } while (0)
#define CU(call)                                                                            \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            fprintf(stderr, "%s -> %s\n", #call, cudaGetErrorString(e_));                   \
            return 3;                                                                       \
        }                                                                                   \
    } while (0)

static void* pool[2 * L];
static unsigned char buf[PIECE];

static unsigned char pattern(uint64_t key, int q, size_t i) {
    return (unsigned char)((key >> (8 * (i % 7))) + (uint64_t)q * 29u + i);
}

/* the engine's part: produce the KV of the flagged blocks */
static int fill(const eakv_turn_view* v) {
    for (int64_t j = 0; j < v->n_blocks; ++j) {
        if (!v->needs_fill[j]) continue;
        for (int q = 0; q < 2 * L; ++q) {
            for (size_t i = 0; i < PIECE; ++i) buf[i] = pattern(v->keys[j], q, i);
            CU(cudaMemcpy((char*)pool[q] + (size_t)v->gpu_block[j] * PIECE, buf, PIECE, cudaMemcpyHostToDevice));
        }
    }
    return 0;
}

static void show(const char* name, const eakv_turn_view* v) {
    printf("%s blocks=%" PRId64 " G=%" PRId64 " H=%" PRId64 " restore=%" PRId64 "..%" PRId64
           " fresh=%" PRId64 " fill=%" PRId64 " store=%" PRId64 " tail=%d\n",
           name, v->n_blocks, v->gpu_prefix_blocks, v->host_prefix_blocks, v->restore_lo, v->restore_hi,
           v->fresh_tokens, v->n_fill, v->n_stored_blocks, v->tail_block >= 0);
}

int main(void) {
    for (int q = 0; q < 2 * L; ++q) {
        CU(cudaMalloc(&pool[q], NB * PIECE));
        CU(cudaMemset(pool[q], 0, NB * PIECE));
    }
    /* prompts live in pinned host memory: the library's kernels read them there */
    int32_t* p1 = NULL;
    int32_t* p2 = NULL;
    CU(cudaHostAlloc((void**)&p1, 7 * B * sizeof(int32_t), cudaHostAllocDefault));
    CU(cudaHostAlloc((void**)&p2, 8 * B * sizeof(int32_t), cudaHostAllocDefault));
    for (int i = 0; i < 7 * B; ++i) p1[i] = (int32_t)(((uint32_t)i * 2246822519u) % 40000u);
    for (int i = 0; i < 8 * B; ++i) p2[i] = (int32_t)(((uint32_t)i * 3266489917u) % 40000u) + 40000;

    eakv_config cfg;
    CK(eakv_config_init(&cfg));
    cfg.num_layers = L; cfg.kv_heads = HEADS; cfg.head_dim = DIM; cfg.block_size = B; cfg.elem_bytes = ELEM;
    cfg.gpu_blocks = NB; cfg.host_blocks = KH;
    cfg.kv_base = pool;
    eakv_ctx* ctx = NULL;
    CK(eakv_create(&cfg, &ctx));

    eakv_turn_view v;
    uint64_t keys1[6];
    CK(eakv_turn_begin(ctx, p1, 6 * B + 4, NULL, 0, 1, 1000, NULL, &v));
    show("turn1", &v);
    memcpy(keys1, v.keys, sizeof keys1);
    if (fill(&v)) return 3;
    CK(eakv_turn_end(ctx, NULL));

    CK(eakv_turn_begin(ctx, p2, 8 * B, NULL, 0, 2, 2000, NULL, &v));
    show("turn2", &v);
    if (fill(&v)) return 3;
    CK(eakv_turn_end(ctx, NULL));

    /* the first prompt again, one block longer; its known keys are passed in, the new block is hashed */
    CK(eakv_turn_begin(ctx, p1, 7 * B, keys1, 6, 1, 3000, NULL, &v));
    show("turn3", &v);
    CK(eakv_sync(ctx));
    int ok = 1;
    for (int64_t j = v.restore_lo; j < v.restore_hi; ++j) {
        for (int q = 0; q < 2 * L; ++q) {
            CU(cudaMemcpy(buf, (char*)pool[q] + (size_t)v.gpu_block[j] * PIECE, PIECE, cudaMemcpyDeviceToHost));
            for (size_t i = 0; i < PIECE; ++i)
                if (buf[i] != pattern(v.keys[j], q, i)) { ok = 0; break; }
        }
    }
    printf("restored %s\n", ok ? "ok" : "BAD");
    printf("key7 %016" PRIx64 "\n", v.keys[6]);
    if (fill(&v)) return 3;
    CK(eakv_turn_end(ctx, NULL));
    CK(eakv_destroy(ctx));
    for (int q = 0; q < 2 * L; ++q) cudaFree(pool[q]);
    cudaFreeHost(p1);
    cudaFreeHost(p2);
    return ok ? 0 : 1;
}
