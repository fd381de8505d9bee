/*
 * CPU oracle for the shared-memory exchange microkernel -- TEST INFRASTRUCTURE, not part of the
 * product. Plain loops, no blocking, no vector code; nothing here is shared with the CUDA path.
 *
 * The operation (the paper names a shared-memory benchmark with a repetition count in Table 1 but
 * gives no definition of it; this is the definition this repository uses):
 *   - the n 32-bit words are cut into tiles of 8 rows x 1024 columns, row-major (8192 words);
 *   - one round replaces, in every tile, row k by row k + row ((k + 1) mod 8) + row ((k + 2) mod 8),
 *     all eight rows taken from the values before the round, addition modulo 2^32;
 *   - a word past the last whole tile is a one-row tile of its own (its cyclic neighbours are the
 *     word itself): one round replaces w by w + w + w;
 *   - out = the array after `rounds` rounds.
 * The round is a bijection on the words of a tile (1 + x + x^2 is a unit modulo x^8 - 1 and 2^32,
 * and 3 is odd), so no number of rounds loses the input: the paper's repetition counts (Table 1:
 * 300 to 1500, default 600) all give outputs that depend on every input word and on the count.
 */
#include <pthread.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ROWS = 8, COLS = 1024, TILE = ROWS * COLS };

static void mix_tile(const uint32_t *x, uint32_t *out, unsigned rounds) {
    static _Thread_local uint32_t cur[ROWS][COLS], nxt[ROWS][COLS];
    memcpy(cur, x, sizeof cur);
    for (unsigned r = 0; r < rounds; ++r) {
        for (int k = 0; k < ROWS; ++k)
            for (int c = 0; c < COLS; ++c)
                nxt[k][c] = cur[k][c] + cur[(k + 1) % ROWS][c] + cur[(k + 2) % ROWS][c];
        memcpy(cur, nxt, sizeof cur);
    }
    memcpy(out, cur, sizeof cur);
}

void oracle_shmem_mix_u32(const uint32_t *x, uint32_t *out, unsigned rounds, size_t n) {
    const size_t tiles = n / TILE;
    for (size_t t = 0; t < tiles; ++t) mix_tile(x + t * TILE, out + t * TILE, rounds);
    for (size_t i = tiles * TILE; i < n; ++i) {
        uint32_t w = x[i];
        for (unsigned r = 0; r < rounds; ++r) w = w + w + w;
        out[i] = w;
    }
}

/* All-cores form: whole tiles are dealt to threads in contiguous ranges; each range is run by
 * the function above (the ragged tail goes with the last range). */
struct piece { const uint32_t *x; uint32_t *out; unsigned rounds; size_t n; };
static void *run_piece(void *p) {
    struct piece *q = (struct piece *)p;
    oracle_shmem_mix_u32(q->x, q->out, q->rounds, q->n);
    return NULL;
}
int oracle_shmem_mix_u32_mt(const uint32_t *x, uint32_t *out, unsigned rounds, size_t n, int nthreads) {
    if (nthreads < 1) nthreads = 1;
    const size_t tiles = n / TILE;
    if ((size_t)nthreads > tiles) nthreads = tiles ? (int)tiles : 1;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    struct piece *pc = (struct piece *)malloc(sizeof(struct piece) * (size_t)nthreads);
    if (!th || !pc) { free(th); free(pc); return 1; }
    const size_t per = tiles / (size_t)nthreads, extra = tiles % (size_t)nthreads;
    size_t t0 = 0;
    for (int i = 0; i < nthreads; ++i) {
        const size_t cnt = per + ((size_t)i < extra ? 1 : 0);
        pc[i].x = x + t0 * TILE; pc[i].out = out + t0 * TILE; pc[i].rounds = rounds;
        pc[i].n = (i == nthreads - 1) ? n - t0 * TILE : cnt * TILE;
        t0 += cnt;
        if (pthread_create(&th[i], NULL, run_piece, &pc[i]) != 0) {
            for (int j = 0; j < i; ++j) pthread_join(th[j], NULL);      /* they still use pc[] */
            free(th); free(pc);
            return 2;
        }
    }
    for (int i = 0; i < nthreads; ++i) pthread_join(th[i], NULL);
    free(th); free(pc);
    return 0;
}
