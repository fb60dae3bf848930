/* The library used from plain C (compiled as C99 by tests/test_library_abi.py): a schedule-only timeline whose
 * schedule dump is printed and compared with the one the Python binding gets for the same calls. */
#include "hpl.h"
#include <stdio.h>
#include <string.h>
int main(void) {
    hpl_config cfg; memset(&cfg, 0, sizeof cfg);
    cfg.chunk_bytes = 64; cfg.reduce_degree = 2; cfg.bcast_degree = 2; cfg.fuse = 1;
    hpl_ctx* c = 0;
    if (hpl_init(&cfg, 0, &c) != HPL_OK) return 1;
    int64_t ids[3] = {1, 2, 3};
    for (int i = 0; i < 3; ++i) if (hpl_create(c, ids[i], i, 256, HPL_F32) != HPL_OK) return 2;
    if (hpl_reduce(c, 9, ids, 3, 2, HPL_SUM, HPL_F32) != HPL_OK) return 3;
    hpl_advance(c, 10); hpl_put(c, 2, (const void*)4096, 256);
    hpl_advance(c, 20); hpl_put(c, 3, (const void*)8192, 128);
    int64_t words[256]; size_t n = 0;
    if (hpl_schedule_dump(c, 9, words, 256, &n) != HPL_OK) return 4;
    for (size_t i = 0; i < n; ++i) printf("%lld ", (long long)words[i]);
    printf("\n");
    hpl_stats_t st; hpl_stats(c, &st);
    printf("%s\n", hpl_strerror(HPL_ERR_TIMEOUT));
    return hpl_shutdown(c);
}
