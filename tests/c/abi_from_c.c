/* The public header must be plain C and the library must link from C: this
 * program includes gk.h in C11 mode, calls the entry points that need no GPU and
 * takes the address of every other one. */
#include <stdio.h>

#include "../../include/gk.h"

int main(void)
{
    gk_geom g = {32, 8, 128, 16, GK_BF16, 0, 0, 0};
    uint64_t bytes = 0;
    uint32_t pages = 0;
    if (gk_blob_size(&g, 4096, &bytes, &pages) != GK_OK) return 1;
    if (bytes != (512ull << 20) || pages != 256) return 2;
    g.dtype = 9;
    if (gk_blob_size(&g, 4096, &bytes, &pages) != GK_ERR_UNSUPPORTED) return 3;
    typedef void (*any_fn)(void);
    any_fn fns[] = {(any_fn)gk_ctx_create, (any_fn)gk_ctx_destroy, (any_fn)gk_last_error, (any_fn)gk_pack,
                    (any_fn)gk_pack_batch, (any_fn)gk_pack_host, (any_fn)gk_page_checksums,
                    (any_fn)gk_page_checksums_noalloc, (any_fn)gk_restore, (any_fn)gk_restore_host,
                    (any_fn)gk_verify, (any_fn)gk_commit, (any_fn)gk_get_stats, (any_fn)gk_ctx_set_tuning,
                    (any_fn)gk_get_kernel_times, (any_fn)gk_restore_stream, (any_fn)gk_fingerprints,
                    (any_fn)gk_blob_digests, (any_fn)gk_pack_layerwise, (any_fn)gk_pack_layerwise_host,
                    (any_fn)gk_restore_layerwise, (any_fn)gk_restore_layerwise_host};
    for (unsigned i = 0; i < sizeof(fns) / sizeof(fns[0]); ++i)
        if (!fns[i]) return 4;
    printf("abi ok: %u entry points\n", (unsigned)(sizeof(fns) / sizeof(fns[0])) + 1u);
    return 0;
}
