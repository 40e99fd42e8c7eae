/* The boundary seen from plain C: the header compiles as C99 and the host-only entry points
 * (no GPU, no context) can be called from a program that links nothing but the library.
 * Built and run by tests/test_cabi_c.py; exits 0 when every check holds. */
#include <stdio.h>
#include <string.h>

#include "kvrebuild.h"

#define CHECK(cond)                                                         \
    do {                                                                    \
        if (!(cond)) {                                                      \
            fprintf(stderr, "check failed at line %d: %s\n", __LINE__, #cond); \
            return 1;                                                       \
        }                                                                   \
    } while (0)

int main(void) {
    /* two requests of 20 and 33 tokens, block size 16: 2 and 3 blocks */
    int32_t lens[2] = {20, 33};
    int32_t tables[2][3] = {{4, 1, -1}, {0, 2, 5}};
    int32_t tokens[53];
    int32_t skip[2] = {-1, -1};
    int64_t computed = -1, chunks = -1, tiles = -1;
    int i;
    for (i = 0; i < 53; ++i) tokens[i] = i % 7;

    CHECK(strcmp(kv_status_str(KVR_OK), kv_status_str(KVR_ERR_BLOCK_OOB)) != 0);
    CHECK(kv_check_inputs(tokens, lens, &tables[0][0], 2, 3, 16, 6, 7) == KVR_OK);
    CHECK(kv_check_inputs(tokens, lens, &tables[0][0], 2, 3, 16, 5, 7) == KVR_ERR_BLOCK_OOB);  /* block 5 of 5 */
    CHECK(kv_check_inputs(tokens, lens, &tables[0][0], 2, 3, 16, 6, 6) == KVR_ERR_TOKEN_OOB);  /* token 6 of 6 */
    tables[1][2] = -1;
    CHECK(kv_check_inputs(tokens, lens, &tables[0][0], 2, 3, 16, 6, 7) == KVR_ERR_TABLE_TOO_SHORT);
    tables[1][2] = 4;   /* request 0's block 0 at another logical index */
    CHECK(kv_check_inputs(tokens, lens, &tables[0][0], 2, 3, 16, 6, 7) == KVR_ERR_ALIAS_CONFLICT);
    tables[1][2] = 5;

    /* plan: nothing shared, chunks of 32 tokens -> 53 computed tokens in 2 chunks */
    CHECK(kv_plan_host(lens, NULL, &tables[0][0], 2, 3, 16, 0, 32, 64, skip, &computed, &chunks, &tiles) == KVR_OK);
    CHECK(skip[0] == 0 && skip[1] == 0 && computed == 53 && chunks == 2 && tiles >= 2);

    /* tensor-parallel partition of a 28/4-head model over two ranks: whole GQA groups, half the columns */
    {
        kv_model_desc full, local;
        kv_tp_shard shard;
        memset(&full, 0, sizeof full);
        full.n_layers = 2; full.d_model = 3584; full.n_q_heads = 28; full.n_kv_heads = 4; full.head_dim = 128;
        full.ffn = 18944; full.vocab = 1024; full.rms_eps = 1e-6f; full.rope_base = 10000.0f; full.dtype = KVR_BF16;
        CHECK(kv_tp_plan_host(&full, 2, 1, &local, &shard) == KVR_OK);
        CHECK(local.n_q_heads == 14 && local.n_kv_heads == 2 && local.ffn == 9472 && local.d_model == 3584);
        CHECK(shard.q_head0 == 14 && shard.kv_head0 == 2 && shard.ffn0 == 9472);
        CHECK(kv_tp_plan_host(&full, 3, 0, &local, &shard) != KVR_OK);   /* 4 kv heads do not split in three */
    }
    printf("c abi host calls ok\n");
    return 0;
}
