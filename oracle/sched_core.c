/*
 * ORACLE (test infrastructure, CPU only).  Plain single-threaded C for the integer / fp64
 * side of the straggler-SGD simulation: the counter-based random stream, the deterministic
 * exponential delay, the minibatch index draw and the arrival process of the four SGD
 * variants.  Nothing here is used by, or shares code with, the CUDA library; only tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Build: gcc -O2 -ffp-contract=off -shared -fPIC (contraction must stay off so that every
 * fp64 operation below is exactly the IEEE operation that is written).
 *
 * What each function follows:
 *   ora_philox4x32_10      Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11)
 *   ora_neg_log_uniform    E = -ln(u) for u = (2k+1)/2^53, a fixed sequence of IEEE operations
 *   ora_delay              X = Delta + E/mu: per-minibatch compute time, i.i.d. over workers and
 *                          minibatches (Section 3.1, modelling assumptions; Exp(mu) has mean 1/mu,
 *                          Corollary 1; shifted exponential of Lemma 4)
 *                          Pareto with shape 2 and scale x_m (the heavy-tailed law of the paper's
 *                          runtime simulations, Figs. 4-5): X = x_m / sqrt(u), P(X > x) = (x_m/x)^2
 *   ora_minibatch_indices  m uniform draws with replacement from the n samples (Section 2)
 *   ora_schedule_*         Section 2.2: K-sync, K-batch-sync, K-async, K-batch-async, with K
 *                          possibly raised at wall-clock checkpoints (Algorithm 1's interval
 *                          structure, doubling rule)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORA_EXPORT __attribute__((visibility("default")))

enum { ORA_KSYNC = 0, ORA_KBATCHSYNC = 1, ORA_KASYNC = 2, ORA_KBATCHASYNC = 3 };
enum { ORA_DELAY_EXP = 0, ORA_DELAY_SHIFTED_EXP = 1, ORA_DELAY_PARETO2 = 2 };

/* ------------------------------------------------------------------------------------------
 * Philox4x32-10.  One round: the 32x32->64 products of counter words 0 and 2 with the two
 * fixed multipliers; the new counter is (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0).  The key is
 * advanced by the two Weyl constants between rounds (not after the last one).
 * ---------------------------------------------------------------------------------------- */
ORA_EXPORT void ora_philox4x32_10(const uint32_t key[2], const uint32_t ctr[4], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Counter layout of the simulation's streams: word 0 = (tag << 24) | chunk, word 1 = the
 * worker's task sequence number, word 2 = worker id, word 3 = global replica id; the key is the
 * 64-bit seed.  tag 0 = delay (chunk 0), tag 1 = minibatch indices (chunk c -> draws 4c..4c+3). */
static void stream_words(uint64_t seed, uint32_t tag, uint32_t chunk, uint32_t replica,
                         uint32_t worker, uint32_t seq, uint32_t out[4]) {
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { (tag << 24) | chunk, seq, worker, replica };
    ora_philox4x32_10(key, ctr, out);
}

/* ------------------------------------------------------------------------------------------
 * E = -ln(u), u = n / 2^53 with n = 2k+1 odd, k the top 52 bits of (x0:x1).
 *   n = f * 2^b, f in [1,2); if f > sqrt(2) halve f and raise b, so f in (sqrt(1/2), sqrt(2)].
 *   ln f = 2 atanh(s), s = (f-1)/(f+1); atanh(s)/s = sum_i s^(2i)/(2i+1), 12 terms, Horner
 *   with fused multiply-adds (|s| <= 0.1716, the dropped tail is below 2e-20).
 *   -ln u = (53 - b) ln 2 - ln f, one fused multiply-add.
 * Every step is an integer operation or one correctly rounded fp64 operation, so the value is a
 * definition that any IEEE machine reproduces bit for bit.
 * ---------------------------------------------------------------------------------------- */
ORA_EXPORT double ora_neg_log_uniform(uint32_t x0, uint32_t x1) {
    uint64_t k = ((uint64_t)x0 << 20) | ((uint64_t)x1 >> 12);    /* 52 bits */
    uint64_t n = 2u * k + 1u;                                    /* odd, < 2^53 */
    int b = 63 - __builtin_clzll(n);                             /* floor(log2 n) */
    uint64_t mant = (n << (52 - b)) & 0x000FFFFFFFFFFFFFull;     /* exact: n has b+1 <= 53 bits */
    uint64_t fbits = 0x3FF0000000000000ull | mant;               /* f in [1,2) */
    if (fbits > 0x3FF6A09E667F3BCDull) {                         /* f > sqrt(2) */
        fbits -= 0x0010000000000000ull;                          /* f/2, exact */
        b += 1;
    }
    double f;
    memcpy(&f, &fbits, sizeof f);
    double s = (f - 1.0) / (f + 1.0);
    double z = s * s;
    double p = 1.0 / 23.0;
    for (int i = 10; i >= 0; --i) p = fma(p, z, 1.0 / (double)(2 * i + 1));
    double lnf = (2.0 * s) * p;
    const double LN2 = 0x1.62e42fefa39efp-1;                     /* bits 0x3FE62E42FEFA39EF */
    return fma((double)(53 - b), LN2, -lnf);
}

/* u = (2k+1) / 2^53 in (0,1), exact in fp64: the same uniform that ora_neg_log_uniform takes the log of */
ORA_EXPORT double ora_uniform(uint32_t x0, uint32_t x1) {
    uint64_t k = ((uint64_t)x0 << 20) | ((uint64_t)x1 >> 12);
    return (double)(2u * k + 1u) * 0x1p-53;
}

ORA_EXPORT double ora_delay(int kind, double mu, double shift, uint64_t seed, uint32_t replica,
                            uint32_t worker, uint32_t seq) {
    uint32_t x[4];
    stream_words(seed, 0u, 0u, replica, worker, seq, x);
    if (kind == ORA_DELAY_PARETO2)          /* shape 2 (given as mu), scale x_m (given as shift) */
        return shift / sqrt(ora_uniform(x[0], x[1]));
    double e = ora_neg_log_uniform(x[0], x[1]);
    double base = (kind == ORA_DELAY_SHIFTED_EXP) ? shift : 0.0;
    return base + e / mu;
}

/* idx_q = floor(u32 * n / 2^32): draw q of the task (replica, worker, seq) is word q%4 of chunk q/4. */
ORA_EXPORT void ora_minibatch_indices(uint64_t seed, uint32_t replica, uint32_t worker,
                                      uint32_t seq, uint64_t n, int32_t m, uint32_t* idx) {
    uint32_t x[4];
    for (int32_t q = 0; q < m; ++q) {
        if (q % 4 == 0) stream_words(seed, 1u, (uint32_t)(q / 4), replica, worker, seq, x);
        idx[q] = (uint32_t)(((uint64_t)x[q % 4] * n) >> 32);
    }
}

/* ------------------------------------------------------------------------------------------
 * Arrival processes.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    int32_t variant;      /* ORA_KSYNC ... */
    int32_t P;            /* workers */
    int32_t K;            /* fixed K (used when t_interval <= 0) */
    int32_t K0;           /* first K of the growing schedule */
    double t_interval;    /* wall-clock length of one interval; <= 0 switches the schedule off */
    int32_t delay_kind;
    double mu, shift;
    uint64_t seed;
} ora_sched_cfg;

/* Per-replica state carried between calls (caller-allocated arrays of length P). */
typedef struct {
    double t;             /* simulated wall clock at the last update */
    int64_t j;            /* number of updates done = current parameter version */
    int32_t started;      /* async variants: 1 once the initial launch at t = 0 happened */
    uint32_t* s;          /* [P] tasks launched so far by each worker */
    uint32_t* tau;        /* [P] version each worker last fetched */
    double* f;            /* [P] absolute finish time of each worker's running task */
} ora_sched_state;

/* K in force for an update that starts at wall-clock t: K0 doubled once per elapsed interval,
 * capped at P. */
static int32_t k_at(const ora_sched_cfg* c, double t) {
    if (!(c->t_interval > 0.0)) return c->K;
    double q = floor(t / c->t_interval);
    int32_t K = c->K0;
    for (double i = 0.0; i < q && K < c->P; i += 1.0) K *= 2;
    return K < c->P ? K : c->P;
}

static double draw(const ora_sched_cfg* c, uint32_t r, int32_t i, uint32_t seq) {
    return ora_delay(c->delay_kind, c->mu, c->shift, c->seed, r, (uint32_t)i, seq);
}

/* index of the smallest (value, worker) among workers not yet taken */
static int32_t argmin_free(const double* v, const uint8_t* taken, int32_t P) {
    int32_t best = -1;
    for (int32_t i = 0; i < P; ++i) {
        if (taken && taken[i]) continue;
        if (best < 0 || v[i] < v[best]) best = i;   /* strict <: the lower id wins a tie */
    }
    return best;
}

/*
 * Advance one replica by `iters` updates.  Outputs are rows of length `iters` (t, K_used) or
 * iters x K_stride (worker, stale, seq), padded with 0xFFFF / 0xFFFFFFFF.
 * Returns 0, or 1 on a bad argument.
 */
ORA_EXPORT int ora_schedule_run(const ora_sched_cfg* c, uint32_t replica, ora_sched_state* st,
                                int64_t iters, int32_t K_stride, double* t_out, uint16_t* K_out,
                                uint16_t* worker_out, uint32_t* stale_out, uint32_t* seq_out) {
    const int32_t P = c->P;
    if (P < 1 || iters < 0 || !(c->mu > 0.0)) return 1;
    double* x = (double*)malloc(sizeof(double) * (size_t)P);
    uint8_t* taken = (uint8_t*)malloc((size_t)P);
    const int async = (c->variant == ORA_KASYNC || c->variant == ORA_KBATCHASYNC);

    if (async && !st->started) {
        /* all workers fetch w_0 and start their first minibatch at t = 0 */
        for (int32_t i = 0; i < P; ++i) {
            st->f[i] = 0.0 + draw(c, replica, i, st->s[i]);
            st->s[i] += 1;
            st->tau[i] = 0;
        }
        st->started = 1;
    }

    for (int64_t u = 0; u < iters; ++u) {
        const int64_t j = st->j;
        const int32_t K = k_at(c, st->t);
        if (K < 1 || K > P || K > K_stride) { free(x); free(taken); return 1; }
        uint16_t* wk = worker_out + u * K_stride;
        uint32_t* sl = stale_out + u * K_stride;
        uint32_t* sq = seq_out + u * K_stride;
        for (int32_t l = 0; l < K_stride; ++l) { wk[l] = 0xFFFFu; sl[l] = 0xFFFFFFFFu; sq[l] = 0xFFFFFFFFu; }

        if (c->variant == ORA_KSYNC) {
            /* every worker starts one minibatch at w_j; the K earliest are used, the rest
             * are cancelled; the iteration lasts X_{K:P} */
            for (int32_t i = 0; i < P; ++i) { x[i] = draw(c, replica, i, st->s[i]); st->s[i] += 1; }
            memset(taken, 0, (size_t)P);
            double T = 0.0;
            for (int32_t l = 0; l < K; ++l) {
                int32_t i = argmin_free(x, taken, P);
                taken[i] = 1;
                wk[l] = (uint16_t)i; sl[l] = 0u; sq[l] = st->s[i] - 1u;
                T = x[i];
            }
            st->t += T;
        } else if (c->variant == ORA_KBATCHSYNC) {
            /* every worker starts at w_j; a finisher pushes and starts another minibatch at the
             * same w_j; the update uses the first K minibatches, everything in flight is dropped */
            for (int32_t i = 0; i < P; ++i) { x[i] = draw(c, replica, i, st->s[i]); st->s[i] += 1; }
            double T = 0.0;
            for (int32_t l = 0; l < K; ++l) {
                int32_t i = argmin_free(x, NULL, P);
                wk[l] = (uint16_t)i; sl[l] = 0u; sq[l] = st->s[i] - 1u;
                T = x[i];
                if (l + 1 < K) { x[i] = x[i] + draw(c, replica, i, st->s[i]); st->s[i] += 1; }
            }
            st->t += T;
        } else if (c->variant == ORA_KASYNC) {
            /* the K earliest finishers contribute gradients taken at the version each last
             * fetched; the others keep computing; the K contributors wait for the update, fetch
             * w_{j+1} and restart together at the update time */
            memset(taken, 0, (size_t)P);
            double tK = 0.0;
            for (int32_t l = 0; l < K; ++l) {
                int32_t i = argmin_free(st->f, taken, P);
                taken[i] = 1;
                wk[l] = (uint16_t)i; sl[l] = (uint32_t)(j - (int64_t)st->tau[i]); sq[l] = st->s[i] - 1u;
                tK = st->f[i];
            }
            st->t = tK;
            for (int32_t l = 0; l < K; ++l) {
                int32_t i = wk[l];
                st->tau[i] = (uint32_t)(j + 1);
                st->f[i] = st->t + draw(c, replica, i, st->s[i]);
                st->s[i] += 1;
            }
        } else { /* ORA_KBATCHASYNC */
            /* every finisher pushes; the K-th push triggers the update; the pusher then fetches
             * whatever the server holds (w_{j+1} for the K-th pusher) and restarts at once */
            for (int32_t l = 0; l < K; ++l) {
                int32_t i = argmin_free(st->f, NULL, P);
                wk[l] = (uint16_t)i; sl[l] = (uint32_t)(j - (int64_t)st->tau[i]); sq[l] = st->s[i] - 1u;
                if (l + 1 == K) { st->t = st->f[i]; st->tau[i] = (uint32_t)(j + 1); }
                else            { st->tau[i] = (uint32_t)j; }
                st->f[i] = st->f[i] + draw(c, replica, i, st->s[i]);
                st->s[i] += 1;
            }
        }
        st->j = j + 1;
        t_out[u] = st->t;
        K_out[u] = (uint16_t)K;
    }
    free(x); free(taken);
    return 0;
}
