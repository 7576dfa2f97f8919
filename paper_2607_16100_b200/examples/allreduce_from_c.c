/* The library from plain C: no Python, no torch, no CUDA header -- only include/symar.h and libsymar.so.
 *
 *   allreduce_from_c P dtype count algo in.bin out.bin
 *
 * reads P rows of `count` elements (dtype 0 = fp32, 1 = bf16; row q is rank q's input) from in.bin,
 * creates a heap that the library owns, runs one AllReduce through the host-buffer entry point and
 * writes every rank's result (P rows again) to out.bin.  Exit code 0 = done and the device status
 * word is clean; anything else names the step that failed on stderr.
 *
 *   gcc -std=c99 -I include allreduce_from_c.c -L <dir of libsymar.so> -lsymar -Wl,-rpath,<dir>
 */
#include <stdio.h>
#include <stdlib.h>

#include "symar.h"

static int fail(const char *what, int rc)
{
    fprintf(stderr, "allreduce_from_c: %s failed (%d)\n", what, rc);
    return 1;
}

int main(int argc, char **argv)
{
    if (argc != 7) {
        fprintf(stderr, "usage: %s P dtype(0=f32,1=bf16) count algo in.bin out.bin\n", argv[0]);
        return 2;
    }
    const int P             = atoi(argv[1]);
    const symar_dtype_t dt  = atoi(argv[2]) ? SYMAR_BF16 : SYMAR_F32;
    const size_t count      = (size_t)strtoull(argv[3], NULL, 10);
    const symar_algo_t algo = (symar_algo_t)atoi(argv[4]);
    const size_t es         = dt == SYMAR_F32 ? 4 : 2;
    const size_t bytes      = count * es;
    /* input at offset 0 of every rank's user region, output behind it on the next SYMAR_ALIGN boundary */
    const size_t out_off    = (bytes + SYMAR_ALIGN - 1) / SYMAR_ALIGN * SYMAR_ALIGN;
    if (P < 1 || count == 0) return fail("arguments", SYMAR_ERR_INVAL);

    void *host_in = malloc((size_t)P * bytes), *host_out = malloc((size_t)P * bytes);
    if (!host_in || !host_out) return fail("malloc", -1);
    FILE *f = fopen(argv[5], "rb");
    if (!f || fread(host_in, bytes, (size_t)P, f) != (size_t)P) return fail("reading the input file", -1);
    fclose(f);

    symheap_t *heap = NULL;
    int rc = symheap_create(&heap, P, out_off + bytes);
    if (rc != SYMAR_OK) return fail("symheap_create", rc);
    void *in  = symheap_rank_ptr(heap, 0, 0);
    void *out = symheap_rank_ptr(heap, 0, out_off);
    if (!in || !out) return fail("symheap_rank_ptr", SYMAR_ERR_INVAL);

    rc = allreduce_host(heap, host_in, host_out, in, out, count, dt, algo, NULL);
    if (rc != SYMAR_OK) return fail("allreduce_host", rc);
    int code = -1, rank = -1, peer = -1, cta = -1;
    rc = symheap_status(heap, &code, &rank, &peer, &cta);       /* synchronous: the stream has drained */
    if (rc != SYMAR_OK) return fail("symheap_status", rc);
    if (code != SYMAR_OK) {
        fprintf(stderr, "allreduce_from_c: device status %d (rank %d, peer %d, CTA slot %d)\n", code, rank, peer, cta);
        return 1;
    }
    symar_algo_t used;
    int ctas = 0, threads = 0;
    if (symar_last_choice(heap, &used, &ctas, &threads) == SYMAR_OK)
        printf("algorithm %d, %d CTAs per rank x %d threads\n", (int)used, ctas, threads);

    f = fopen(argv[6], "wb");
    if (!f || fwrite(host_out, bytes, (size_t)P, f) != (size_t)P) return fail("writing the output file", -1);
    fclose(f);
    rc = symheap_destroy(heap);
    if (rc != SYMAR_OK) return fail("symheap_destroy", rc);
    free(host_in);
    free(host_out);
    return 0;
}
