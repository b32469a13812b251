/* A client of the C boundary written in plain C: no Python, no torch in the process.
 *
 * One agent turn with the five calls (hash, match, tier step, store, load) on a tiny KV shape,
 * then the same prompt again (now a host hit).  Prints what a test compares with the CPU oracle:
 *   keys <hex> ...        block keys of the prompt
 *   match1 G H / match2 G H
 *   step admitted=<n> slots=<s0,s1,...>
 *   roundtrip ok|BAD      bytes restored into other pool blocks equal the bytes stored
 *   untouched ok|BAD      no other pool block changed
 * Exit code 0 when every call returned EAKV_OK and both byte checks passed.
 *
 * Build: gcc -std=c99 five_calls.c -I<repo>/include -I<cuda>/include -L<pkg> -leakv -L<cuda>/lib64 -lcudart
 */
#include <cuda_runtime_api.h>
#include <inttypes.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "eakv.h"

enum { L = 2, HEADS = 2, DIM = 64, B = 16, ELEM = 2, NB = 64, KH = 32, NTOK = 100 };
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

static unsigned char pattern(int q, int blk, size_t i) {
    return (unsigned char)((q * 131 + blk * 31 + (int)(i % 251) * 7 + (int)(i / 251)) & 0xff);
}

int main(void) {
    void* pool[2 * L];
    unsigned char* host = (unsigned char*)malloc(NB * PIECE);
    unsigned char* back = (unsigned char*)malloc(NB * PIECE);
    if (!host || !back) return 4;
    for (int q = 0; q < 2 * L; ++q) {
        for (int blk = 0; blk < NB; ++blk)
            for (size_t i = 0; i < PIECE; ++i) host[blk * PIECE + i] = pattern(q, blk, i);
        CU(cudaMalloc(&pool[q], NB * PIECE));
        CU(cudaMemcpy(pool[q], host, NB * PIECE, cudaMemcpyHostToDevice));
    }

    int32_t tokens[NTOK];
    for (int i = 0; i < NTOK; ++i) tokens[i] = (int32_t)(((uint32_t)i * 2654435761u) % 50000u);
    int32_t* tokens_dev = NULL;
    uint64_t* keys_dev = NULL;
    CU(cudaMalloc((void**)&tokens_dev, sizeof tokens));
    CU(cudaMalloc((void**)&keys_dev, (NTOK / B) * sizeof(uint64_t)));
    CU(cudaMemcpy(tokens_dev, tokens, sizeof tokens, cudaMemcpyHostToDevice));

    eakv_config cfg;
    CK(eakv_config_init(&cfg));
    cfg.num_layers = L; cfg.kv_heads = HEADS; cfg.head_dim = DIM; cfg.block_size = B; cfg.elem_bytes = ELEM;
    cfg.gpu_blocks = NB; cfg.host_blocks = KH;
    cfg.kv_base = pool;
    cfg.policy = EAKV_POLICY_WRITE_ALL;
    eakv_ctx* ctx = NULL;
    CK(eakv_create(&cfg, &ctx));

    /* a1: keys */
    int64_t nblk = 0;
    uint64_t keys[NTOK / B];
    CK(eakv_hash_blocks(ctx, tokens_dev, NTOK, eakv_hash_seed(ctx), keys_dev, &nblk, NULL));
    CU(cudaMemcpy(keys, keys_dev, (size_t)nblk * sizeof(uint64_t), cudaMemcpyDeviceToHost));
    printf("keys");
    for (int64_t j = 0; j < nblk; ++j) printf(" %016" PRIx64, keys[j]);
    printf("\n");

    /* a2: nothing is cached yet */
    int64_t G = -1, H = -1;
    int32_t gpu_ids[NTOK / B], slots[NTOK / B];
    CK(eakv_match(ctx, keys, nblk, &G, &H, gpu_ids, slots));
    printf("match1 %" PRId64 " %" PRId64 "\n", G, H);

    /* a3: bookkeeping and admission */
    uint8_t hit[NTOK / B], admit[NTOK / B];
    uint64_t evk[NTOK / B];
    int32_t evs[NTOK / B];
    int64_t nev = NTOK / B;
    eakv_step_info info;
    CK(eakv_tier_step(ctx, keys, nblk, 7, NTOK, 1000, hit, admit, slots, evk, evs, &nev, &info));
    int admitted = 0;
    printf("step admitted=");
    for (int64_t j = 0; j < nblk; ++j) admitted += admit[j];
    printf("%d slots=", admitted);
    for (int64_t j = 0; j < nblk; ++j) printf("%s%d", j ? "," : "", slots[j]);
    printf("\n");

    /* a5: the prompt's blocks live in pool blocks 10, 11, ... */
    int32_t table[NTOK / B], table2[NTOK / B];
    for (int64_t j = 0; j < nblk; ++j) { table[j] = 10 + (int32_t)j; table2[j] = 40 + 2 * (int32_t)j; }
    CK(eakv_store(ctx, table, admit, slots, nblk, NULL));
    CK(eakv_sync(ctx));

    /* same prompt again: all of it is a host hit; a4 restores it into other blocks */
    CK(eakv_match(ctx, keys, nblk, &G, &H, gpu_ids, slots));
    printf("match2 %" PRId64 " %" PRId64 "\n", G, H);
    CK(eakv_load(ctx, slots, table2, H, NULL));
    CK(eakv_sync(ctx));

    int round_ok = 1, rest_ok = 1;
    for (int q = 0; q < 2 * L; ++q) {
        CU(cudaMemcpy(back, pool[q], NB * PIECE, cudaMemcpyDeviceToHost));
        for (int blk = 0; blk < NB; ++blk) {
            int src = blk;                                   /* untouched blocks keep their own pattern */
            for (int64_t j = 0; j < H; ++j)
                if (table2[j] == blk) src = table[j];
            for (size_t i = 0; i < PIECE; ++i) {
                if (back[blk * PIECE + i] != pattern(q, src, i)) {
                    if (src == blk) rest_ok = 0; else round_ok = 0;
                    break;
                }
            }
        }
    }
    printf("roundtrip %s\n", round_ok ? "ok" : "BAD");
    printf("untouched %s\n", rest_ok ? "ok" : "BAD");

    eakv_stats st;
    CK(eakv_get_stats(ctx, &st));
    printf("stats stored=%" PRId64 " loaded=%" PRId64 "\n", (int64_t)st.blocks_stored, (int64_t)st.blocks_loaded);
    CK(eakv_destroy(ctx));
    for (int q = 0; q < 2 * L; ++q) cudaFree(pool[q]);
    cudaFree(tokens_dev);
    cudaFree(keys_dev);
    free(host);
    free(back);
    return (round_ok && rest_ok) ? 0 : 1;
}
