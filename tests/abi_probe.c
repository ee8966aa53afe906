/* A plain C99 caller of the library: checks that include/h1b.h is valid C and that the entry points link and answer
 * from C without a GPU (size queries and argument checks only; nothing here launches a kernel). */
#include <stdio.h>
#include <string.h>

#include "h1b.h"

int main(void)
{
    h1b_config c;
    memset(&c, 0, sizeof c);
    c.n_layers = 32; c.n_q_heads = 32; c.n_kv_heads = 32; c.head_dim = 128; c.sketch_bits = 128; c.group_size = 32;
    c.max_batch = 1; c.max_seq = 8192; c.device = 0; c.flags = 0;
    if (h1b_entry_bytes(&c) != 96) { printf("entry bytes %lu\n", (unsigned long)h1b_entry_bytes(&c)); return 1; }
    if (h1b_cache_bytes(&c) < (size_t)32 * 32 * 8192 * 96) return 2;
    c.flags = H1B_FLAG_FP16_VALUES;
    if (h1b_entry_bytes(&c) != 16 + 256) return 3;
    c.flags = H1B_FLAG_ROPE;
    if (h1b_cache_bytes(&c) == 0) return 4;
    c.flags = 64u;                                   /* an unknown flag */
    if (h1b_cache_bytes(&c) != 0) return 5;
    if (h1b_free(NULL) != H1B_ERR_NULL) return 6;
    if (h1b_poll_status(NULL) != H1B_ERR_NULL) return 7;
    if (h1b_decode_attention(NULL, 0, 1, NULL, 1.0f, NULL, 1, NULL) != H1B_ERR_NULL) return 8;
    if (h1b_append_kv(NULL, 0, 1, NULL, NULL, NULL, 1, 1, NULL) != H1B_ERR_NULL) return 9;
    {
        h1b_ctx *ctx = NULL;
        c.flags = 0;
        if (h1b_init_projection(&c, 0, NULL, NULL, 0, NULL, &ctx) != H1B_ERR_NULL || ctx != NULL) return 10;
        if (strstr(h1b_last_error(NULL), "workspace") == NULL) return 11;
    }
    if (H1B_MAX_QUERY_TOKENS != 16) return 12;
    printf("ok\n");
    return 0;
}
