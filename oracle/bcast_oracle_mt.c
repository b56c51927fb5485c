/*
 * bcast_oracle_mt.c -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * The CPU baseline on all host cores: replays a schedule that the single-threaded oracle
 * (bcast_oracle.c) produced, with the copies of every step shared out over a team of threads.
 * It computes nothing of the method itself -- which process sends which chunk to whom in which
 * step is read from the schedule -- and exists only so that the benchmark can say what the same
 * memcpy work costs when every core of the host takes part.  The single-threaded oracle stays as
 * it is and remains the reference for parity; a test checks that this replay leaves exactly the
 * buffers the oracle leaves.
 *
 * Steps are kept in the paper's order (Section III-A: scatter level by level, then the ring step
 * by step; Section IV for the tuned ring): all threads meet at a barrier after every step, so no
 * message of step s+1 is read before every message of step s has been written.  Inside a step each
 * thread copies its share (an equal slice of the byte range) of every message; the messages of a
 * step never read what the step writes (the oracle checks that when it builds the schedule).
 *
 * It shares no code with the CUDA library.
 */
#define _POSIX_C_SOURCE 200809L
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

enum { F_PHASE = 0, F_STEP, F_SRC, F_DST, F_CHUNK, F_NCHUNKS, F_OFFSET, F_LEN, F_DEP, F_NFIELDS };

typedef struct {
    int P, nthreads;
    uint8_t *const *buf;
    const int64_t *sched;
    int64_t nsched;
    pthread_barrier_t barrier;
} team_t;

typedef struct {
    team_t *team;
    int tid;
} worker_t;

static void copy_share(const team_t *tm, int tid, const int64_t *rec)
{
    const uint64_t len = (uint64_t)rec[F_LEN], off = (uint64_t)rec[F_OFFSET];
    const uint64_t lo = len * (uint64_t)tid / (uint64_t)tm->nthreads;
    const uint64_t hi = len * ((uint64_t)tid + 1) / (uint64_t)tm->nthreads;
    if (hi > lo) memcpy(tm->buf[rec[F_DST]] + off + lo, tm->buf[rec[F_SRC]] + off + lo, (size_t)(hi - lo));
}

static void *worker(void *arg)
{
    const worker_t *w = (const worker_t *)arg;
    team_t *tm = w->team;
    pthread_barrier_wait(&tm->barrier);                    /* start together */
    int64_t i = 0;
    while (i < tm->nsched) {
        const int64_t phase = tm->sched[i * F_NFIELDS + F_PHASE], step = tm->sched[i * F_NFIELDS + F_STEP];
        for (; i < tm->nsched && tm->sched[i * F_NFIELDS + F_PHASE] == phase && tm->sched[i * F_NFIELDS + F_STEP] == step; i++)
            copy_share(tm, w->tid, tm->sched + i * F_NFIELDS);
        pthread_barrier_wait(&tm->barrier);                /* the step is complete before the next begins */
    }
    return NULL;
}

/*
 * Replay `nsched` schedule records (9 x int64 each: phase, step, src, dst, chunk, nchunks, offset,
 * len, dep; grouped by step, as the oracle writes them) on P host buffers with `nthreads` threads.
 * buf[root] holds the message on entry.  *seconds receives the wall time from the common start to
 * the end of the last step.  Returns 0, or -1 on bad arguments, -2 if threads cannot be created.
 */
int oracle_bcast_replay_mt(int P, uint8_t *const *buf, const int64_t *sched, int64_t nsched, int nthreads, double *seconds)
{
    if (P < 1 || !buf || (!sched && nsched) || nsched < 0 || nthreads < 1 || !seconds) return -1;
    for (int64_t i = 0; i < nsched; i++) {
        const int64_t *r = sched + i * F_NFIELDS;
        if (r[F_SRC] < 0 || r[F_SRC] >= P || r[F_DST] < 0 || r[F_DST] >= P || r[F_LEN] < 0 || r[F_OFFSET] < 0) return -1;
    }
    team_t tm;
    tm.P = P; tm.nthreads = nthreads; tm.buf = buf; tm.sched = sched; tm.nsched = nsched;
    if (pthread_barrier_init(&tm.barrier, NULL, (unsigned)nthreads)) return -2;
    pthread_t *th = malloc(sizeof(pthread_t) * (size_t)nthreads);
    worker_t *ws = malloc(sizeof(worker_t) * (size_t)nthreads);
    if (!th || !ws) { free(th); free(ws); pthread_barrier_destroy(&tm.barrier); return -2; }
    /* the calling thread is member 0 of the team; if a thread cannot be created nothing has started yet
       (everyone waits at the first barrier), so the team is shrunk to what exists */
    int made = 1;
    ws[0].team = &tm; ws[0].tid = 0;
    for (int t = 1; t < nthreads; t++) {
        ws[t].team = &tm; ws[t].tid = t;
        if (pthread_create(&th[t], NULL, worker, &ws[t])) break;
        made++;
    }
    int rc = 0;
    if (made != nthreads) {
        /* cannot run with fewer members than the barrier expects: cancel the waiting ones */
        for (int t = 1; t < made; t++) { pthread_cancel(th[t]); pthread_join(th[t], NULL); }
        rc = -2;
    } else {
        struct timespec t0, t1;
        clock_gettime(CLOCK_MONOTONIC, &t0);
        worker(&ws[0]);
        clock_gettime(CLOCK_MONOTONIC, &t1);
        for (int t = 1; t < nthreads; t++) pthread_join(th[t], NULL);
        *seconds = (double)(t1.tv_sec - t0.tv_sec) + 1e-9 * (double)(t1.tv_nsec - t0.tv_nsec);
    }
    free(th); free(ws);
    pthread_barrier_destroy(&tm.barrier);
    return rc;
}
