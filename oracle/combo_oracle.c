/*
 * CPU oracle for one segmented-gossip synchronization round
 * ("Decentralized Federated Learning: A Segmented Gossip Approach", Section 3
 * and Section 4.1).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded
 * statement of what the round computes, used only to check the CUDA library
 * and to time a CPU baseline.  It shares no code, header, table or constant
 * generator with the CUDA path and the product never calls it.
 *
 * Notation (the paper's): n = N workers, W = flat parameter vector of P
 * entries, S segments, R model replicas, |D_j| = dataset size of worker j,
 * P_l = set of workers providing segment l (the worker itself included).
 *
 * What is pinned by the CPU tests, function by function:
 *   oracle_segment_bounds        closed form + partition property
 *   oracle_splitmix64_next       published splitmix64 output sequence
 *   oracle_rand32                avalanche / range statistics only
 *   oracle_select_peers          invariants Section 4.1 step (2) fixes (never
 *                                self, no repeat, even spread, all distinct
 *                                when S*R <= n-1), uniformity of the shuffle.
 *                                Its exact tables are PARITY UNPINNED by the
 *                                paper, which names no generator.
 *   oracle_select_peers_active   equals oracle_select_peers when all are online;
 *                                never an offline peer; same invariants on the
 *                                online pool; offline rows are -1
 *   oracle_segment_aggregate_members  equals oracle_segment_aggregate without
 *                                newcomers / absent peers; exact rationals with
 *                                them; a newcomer's own values never matter
 *   oracle_divergence            exact rational brute force of Eq. 7 on tiny
 *                                inputs, two-worker closed form, identical
 *                                models (zero), R = n-1 (zero, as the paper
 *                                states), scaling and translation laws
 *   oracle_segment_aggregate_*   exact rational brute force of Eq. 3 on tiny
 *                                inputs, hand-worked dyadic example, R = 0,
 *                                R = n-1 (all-reduce / FedAvg mean), S = 1,
 *                                convexity, identical inputs
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Eq. 1: W = (W[1], ..., W[S]), S non-overlapping segments with the   */
/* same number of parameters.  Reading for P mod S != 0: segment       */
/* length ceil(P/S), the last segment(s) shorter, possibly empty.      */
/* ------------------------------------------------------------------ */
int64_t oracle_segment_length(int64_t P, int S) { return (P + S - 1) / S; }

void oracle_segment_bounds(int64_t P, int S, int64_t *lo, int64_t *hi) {
    int64_t L = oracle_segment_length(P, S);
    for (int l = 0; l < S; ++l) {
        int64_t a = (int64_t)l * L, b = (int64_t)(l + 1) * L;
        lo[l] = a < P ? a : P;
        hi[l] = b < P ? b : P;
    }
}

/* ------------------------------------------------------------------ */
/* Counter-based random numbers.  The paper only says "randomly        */
/* selected"; the generator below is this library's definition:        */
/* splitmix64 (Steele, Lea, Flood, OOPSLA 2014) and a keyed chain of   */
/* its output function over the counter (seed, round|w, epoch|t).      */
/* ------------------------------------------------------------------ */
static uint64_t sm64_mix(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* One step of the splitmix64 generator: advances *state, returns output. */
uint64_t oracle_splitmix64_next(uint64_t *state) {
    *state += 0x9E3779B97F4A7C15ULL;
    return sm64_mix(*state);
}

/* rand32(seed, round, w, e, t): three chained splitmix64 steps, each
 * started from the previous output xor the next counter word; the result
 * is the high half of the last output. */
uint32_t oracle_rand32(uint64_t seed, uint32_t round, uint32_t w, uint32_t e, uint32_t t) {
    uint64_t s = seed;
    uint64_t h = oracle_splitmix64_next(&s);
    s = h ^ (((uint64_t)round << 32) | (uint64_t)w);
    h = oracle_splitmix64_next(&s);
    s = h ^ (((uint64_t)e << 32) | (uint64_t)t);
    h = oracle_splitmix64_next(&s);
    return (uint32_t)(h >> 32);
}

/* ------------------------------------------------------------------ */
/* Section 4.1 step (2): each worker issues S*R pull requests; every   */
/* target is drawn at random from all the OTHER workers without        */
/* replacement until no option is left.  Readings: after the pool is   */
/* exhausted a fresh random order of the others starts (new epoch);    */
/* P_l in Eq. 3 is a set, so a segment never gets one peer twice: the  */
/* peers already chosen for the current segment are moved, in order,   */
/* behind the rest of a freshly shuffled pool.                         */
/* idx layout [w][l][r], each (w,l) row ascending.                     */
/* Returns 0, or 1 for invalid arguments.                              */
/* ------------------------------------------------------------------ */
static int cmp_i32(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int oracle_select_peers(uint64_t seed, uint32_t round, int N, int S, int R, int32_t *idx) {
    if (N < 1 || S < 1 || R < 0 || R > N - 1) return 1;
    if (R == 0) return 0;
    int M = N - 1;
    int32_t *perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)M);
    int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)M);
    int32_t *chosen = (int32_t *)malloc(sizeof(int32_t) * (size_t)R);
    for (int w = 0; w < N; ++w) {
        int pos = M;          /* pool empty: the first draw opens epoch 0 */
        uint32_t epoch = 0;
        int opened = 0;
        for (int l = 0; l < S; ++l) {
            int nc = 0;
            for (int r = 0; r < R; ++r) {
                if (pos == M) {
                    if (opened) ++epoch;
                    opened = 1;
                    /* all the other workers, ascending */
                    for (int i = 0, v = 0; v < N; ++v)
                        if (v != w) perm[i++] = v;
                    /* Fisher-Yates shuffle, t = M-1 down to 1 */
                    for (int t = M - 1; t >= 1; --t) {
                        uint32_t u = oracle_rand32(seed, round, (uint32_t)w, epoch, (uint32_t)t);
                        int j = (int)(((uint64_t)u * (uint64_t)(t + 1)) >> 32);
                        int32_t s = perm[t]; perm[t] = perm[j]; perm[j] = s;
                    }
                    /* peers this segment already has go to the back, stably */
                    if (nc > 0) {
                        int a = 0;
                        for (int i = 0; i < M; ++i) {
                            int taken = 0;
                            for (int c = 0; c < nc; ++c) taken |= (chosen[c] == perm[i]);
                            if (!taken) tmp[a++] = perm[i];
                        }
                        for (int i = 0; i < M; ++i) {
                            int taken = 0;
                            for (int c = 0; c < nc; ++c) taken |= (chosen[c] == perm[i]);
                            if (taken) tmp[a++] = perm[i];
                        }
                        memcpy(perm, tmp, sizeof(int32_t) * (size_t)M);
                    }
                    pos = 0;
                }
                chosen[nc++] = perm[pos++];
            }
            qsort(chosen, (size_t)R, sizeof(int32_t), cmp_i32);
            memcpy(idx + ((size_t)w * S + l) * R, chosen, sizeof(int32_t) * (size_t)R);
        }
    }
    free(perm); free(tmp); free(chosen);
    return 0;
}

/* ------------------------------------------------------------------ */
/* bf16 <-> binary32/binary64 (bf16 = the upper 16 bits of binary32).  */
/* ------------------------------------------------------------------ */
static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f; memcpy(&f, &u, 4); return f;
}

/* round-to-nearest-even binary32 -> bf16 (finite inputs) */
uint16_t oracle_f32_to_bf16_rne(float f) {
    uint32_t u; memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------ */
/* Eq. 3 and Eq. 4, evaluated as written, in binary64:                 */
/*   out[w][p] = sum_{j in P_l} |D_j| x_j[p]  /  sum_{j in P_l} |D_j|  */
/* with l the segment holding p and P_l = {w} U idx[w][l][0..R).       */
/* x_j[p] is the value worker j SENDS: its locally updated model       */
/* (Section 4.1 steps 1 and 3), i.e. in[j][p] - lr*grads[j][p] when    */
/* grads is given, in[j][p] otherwise.                                 */
/*                                                                     */
/* `in`/`grads` point at a slab [N][pitch] whose column 0 is global    */
/* column p_begin; columns [p_begin, p_end) are evaluated and written  */
/* to out as [N][p_end-p_begin] doubles.  elem = 4: binary32 input,    */
/* elem = 2: bf16 input.  weights == NULL means |D_j| = 1 for all j.   */
/* ------------------------------------------------------------------ */
static double load_x(const void *base, int elem, size_t off) {
    if (elem == 4) return (double)((const float *)base)[off];
    return (double)bf16_to_f32(((const uint16_t *)base)[off]);
}

int oracle_segment_aggregate(const void *in, const void *grads, double lr, int elem,
                             int64_t pitch, const float *weights, const int32_t *idx,
                             int N, int64_t P, int S, int R,
                             int64_t p_begin, int64_t p_end, double *out) {
    if (N < 1 || P < 1 || S < 1 || R < 0 || R > N - 1) return 1;
    if (p_begin < 0 || p_end > P || p_begin > p_end) return 1;
    if (elem != 4 && elem != 2) return 1;
    int64_t L = oracle_segment_length(P, S);
    int64_t width = p_end - p_begin;
    for (int w = 0; w < N; ++w) {
        for (int64_t p = p_begin; p < p_end; ++p) {
            int l = (int)(p / L);
            const int32_t *peers = idx ? idx + ((size_t)w * S + l) * R : NULL;
            double num = 0.0, den = 0.0;
            for (int m = -1; m < R; ++m) {
                int j = (m < 0) ? w : peers[m];
                size_t off = (size_t)j * (size_t)pitch + (size_t)(p - p_begin);
                double x = load_x(in, elem, off);
                if (grads) x = x - lr * load_x(grads, elem, off);
                double D = weights ? (double)weights[j] : 1.0;
                num += D * x;
                den += D;
            }
            out[(size_t)w * (size_t)width + (size_t)(p - p_begin)] = num / den;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* The same round in binary32 with one fixed operation order, Eq. 3 as */
/* it is written: provider order is self first, then peers ascending;  */
/*   num = |D_self|*x_self, num = fma(|D_j|, x_j, num)                 */
/*   den = |D_self|, den = den + |D_j|            (the same order)     */
/*   out = num * (1/den)      (the reciprocal rounded to binary32)     */
/* With a single provider the quotient is that provider's value and is */
/* taken as such (out = x: R = 0 is the identity, bit for bit).  With  */
/* weights == NULL every |D_j| is 1, the products are exact and num is */
/* the plain sum in that order.  The local step is x = fma(-lr, g, x)  */
/* rounded to binary32.  A bf16 result is the binary32 result rounded  */
/* to nearest even.  This is a                                         */
/* second, tighter yardstick for a binary32 implementation that uses   */
/* the same order; it is itself pinned against the binary64 form.      */
/* out: [N][p_end-p_begin] of float (elem 4) or uint16 bf16 (elem 2).  */
/* ------------------------------------------------------------------ */
int oracle_segment_aggregate_ordered_f32(const void *in, const void *grads, float lr, int elem,
                                         int64_t pitch, const float *weights, const int32_t *idx,
                                         int N, int64_t P, int S, int R,
                                         int64_t p_begin, int64_t p_end, void *out) {
    if (N < 1 || P < 1 || S < 1 || R < 0 || R > N - 1) return 1;
    if (p_begin < 0 || p_end > P || p_begin > p_end) return 1;
    if (elem != 4 && elem != 2) return 1;
    if (grads && elem != 4) return 1;
    int64_t L = oracle_segment_length(P, S);
    int64_t width = p_end - p_begin;
    for (int w = 0; w < N; ++w) {
        for (int l = 0; l < S; ++l) {
            int64_t a = (int64_t)l * L, b = a + L;
            if (a < p_begin) a = p_begin;
            if (b > p_end) b = p_end;
            if (a >= b) continue;
            const int32_t *peers = idx ? idx + ((size_t)w * S + l) * R : NULL;
            volatile float den = weights ? weights[w] : 1.0f;
            for (int r = 0; r < R; ++r) den = den + (weights ? weights[peers[r]] : 1.0f);
            volatile float rden = 1.0f / den;
            for (int64_t p = a; p < b; ++p) {
                float acc = 0.0f;
                for (int m = -1; m < R; ++m) {
                    int j = (m < 0) ? w : peers[m];
                    size_t off = (size_t)j * (size_t)pitch + (size_t)(p - p_begin);
                    float x = (elem == 4) ? ((const float *)in)[off]
                                          : bf16_to_f32(((const uint16_t *)in)[off]);
                    if (grads) x = fmaf(-lr, ((const float *)grads)[off], x);
                    float D = weights ? weights[j] : 1.0f;
                    if (m < 0) { volatile float prod = D * x; acc = (R == 0) ? x : prod; }
                    else acc = fmaf(D, x, acc);
                }
                if (R > 0) { volatile float q = acc * rden; acc = q; }
                size_t o = (size_t)w * (size_t)width + (size_t)(p - p_begin);
                if (elem == 4) ((float *)out)[o] = acc;
                else ((uint16_t *)out)[o] = oracle_f32_to_bf16_rne(acc);
            }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Aggregation divergence (Section 4.3, Definition 2, Eq. 7):          */
/*   rho_i = || W_{t,i} - W_t ||                                       */
/* W_{t,i}: the model worker i holds (row i of `models`); W_t: the     */
/* aggregation of ALL workers, the FedAvg result                       */
/*   W_t = sum_j |D_j| W_j / sum_j |D_j|                               */
/* taken over the rows of `mean_of` (the models the round started      */
/* from; the same array as `models` when mean_of == NULL).  Reading:   */
/* the norm is the Euclidean one.  Binary64 throughout.                */
/* models, mean_of: [N][P] dense, elem 4 = binary32, 2 = bf16.         */
/* ------------------------------------------------------------------ */
int oracle_divergence(const void *models, const void *mean_of, int elem, const float *weights,
                      int N, int64_t P, double *rho) {
    if (N < 1 || P < 1 || (elem != 4 && elem != 2)) return 1;
    if (!mean_of) mean_of = models;
    double den = 0.0;
    for (int j = 0; j < N; ++j) den += weights ? (double)weights[j] : 1.0;
    for (int i = 0; i < N; ++i) rho[i] = 0.0;
    for (int64_t p = 0; p < P; ++p) {
        double num = 0.0;
        for (int j = 0; j < N; ++j)
            num += (weights ? (double)weights[j] : 1.0) * load_x(mean_of, elem, (size_t)j * (size_t)P + (size_t)p);
        double mean = num / den;
        for (int i = 0; i < N; ++i) {
            double d = load_x(models, elem, (size_t)i * (size_t)P + (size_t)p) - mean;
            rho[i] += d * d;
        }
    }
    for (int i = 0; i < N; ++i) rho[i] = sqrt(rho[i]);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Dynamic workers (Section 4.2).                                      */
/* (1) A worker that is offline is not pulled from: requests go to     */
/*     "another worker", so the pool of a worker is the ONLINE others. */
/*     Offline workers issue no requests: their rows are filled -1.    */
/*     With every worker online this is oracle_select_peers exactly.   */
/*     active: N bytes, non-zero = online; NULL = all online.          */
/*     Requires R <= (number of online workers) - 1.                   */
/* ------------------------------------------------------------------ */
int oracle_select_peers_active(uint64_t seed, uint32_t round, int N, int S, int R,
                               const uint8_t *active, int32_t *idx) {
    if (N < 1 || S < 1 || R < 0) return 1;
    int n_on = 0;
    for (int v = 0; v < N; ++v) n_on += (!active || active[v]) ? 1 : 0;
    if (R > 0 && R > n_on - 1) return 1;
    if (R == 0) return 0;
    int32_t *pool = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    int32_t *perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    int32_t *chosen = (int32_t *)malloc(sizeof(int32_t) * (size_t)R);
    for (int w = 0; w < N; ++w) {
        int32_t *rows = idx + (size_t)w * S * R;
        if (active && !active[w]) {
            for (int i = 0; i < S * R; ++i) rows[i] = -1;
            continue;
        }
        int M = 0;
        for (int v = 0; v < N; ++v)
            if (v != w && (!active || active[v])) pool[M++] = v;
        int pos = M;
        uint32_t epoch = 0;
        int opened = 0;
        for (int l = 0; l < S; ++l) {
            int nc = 0;
            for (int r = 0; r < R; ++r) {
                if (pos == M) {
                    if (opened) ++epoch;
                    opened = 1;
                    memcpy(perm, pool, sizeof(int32_t) * (size_t)M);
                    for (int t = M - 1; t >= 1; --t) {
                        uint32_t u = oracle_rand32(seed, round, (uint32_t)w, epoch, (uint32_t)t);
                        int j = (int)(((uint64_t)u * (uint64_t)(t + 1)) >> 32);
                        int32_t s = perm[t]; perm[t] = perm[j]; perm[j] = s;
                    }
                    if (nc > 0) {
                        int a = 0;
                        for (int pass = 0; pass < 2; ++pass)
                            for (int i = 0; i < M; ++i) {
                                int taken = 0;
                                for (int c = 0; c < nc; ++c) taken |= (chosen[c] == perm[i]);
                                if (taken == pass) tmp[a++] = perm[i];
                            }
                        memcpy(perm, tmp, sizeof(int32_t) * (size_t)M);
                    }
                    pos = 0;
                }
                chosen[nc++] = perm[pos++];
            }
            qsort(chosen, (size_t)R, sizeof(int32_t), cmp_i32);
            memcpy(rows + (size_t)l * R, chosen, sizeof(int32_t) * (size_t)R);
        }
    }
    free(pool); free(perm); free(tmp); free(chosen);
    return 0;
}

/* ------------------------------------------------------------------ */
/* (2) Eq. 3 with the provider sets Section 4.2 allows:                */
/*     P_l(w) = ({w} unless w is a newcomer) U {idx[w][l][r] >= 0}.    */
/*     A newcomer has no model of its own yet, so its aggregate is     */
/*     formed from the pulled segments alone; a negative idx entry is  */
/*     a pull that found no online peer.  An empty P_l leaves the      */
/*     worker's own values (reading: nothing to aggregate).            */
/*     newcomer: N bytes or NULL.  mode 0: binary64, quotient of sums, */
/*     out = double; mode 1: the fixed-order binary32 form, out =      */
/*     float (elem 4) or bf16 bits (elem 2).                           */
/* ------------------------------------------------------------------ */
int oracle_segment_aggregate_members(const void *in, int elem, const float *weights, const int32_t *idx,
                                     const uint8_t *newcomer, int N, int64_t P, int S, int R, int mode,
                                     void *out) {
    if (N < 1 || P < 1 || S < 1 || R < 0 || (elem != 4 && elem != 2)) return 1;
    int64_t L = oracle_segment_length(P, S);
    int *prov = (int *)malloc(sizeof(int) * (size_t)(R + 1));
    for (int w = 0; w < N; ++w) {
        for (int l = 0; l < S; ++l) {
            int64_t a = (int64_t)l * L, b = a + L;
            if (b > P) b = P;
            if (a >= b) continue;
            int np = 0;
            if (!newcomer || !newcomer[w]) prov[np++] = w;
            for (int r = 0; r < R; ++r) {
                int k = idx[((size_t)w * S + l) * R + r];
                if (k >= 0) prov[np++] = k;
            }
            if (np == 0) prov[np++] = w;
            volatile float rden32 = 1.0f;
            if (mode == 1) {
                volatile float den = 0.0f;
                for (int q = 0; q < np; ++q) {
                    float D = weights ? weights[prov[q]] : 1.0f;
                    den = (q == 0) ? D : den + D;
                }
                rden32 = 1.0f / den;
            }
            for (int64_t p = a; p < b; ++p) {
                size_t o = (size_t)w * (size_t)P + (size_t)p;
                if (mode == 0) {
                    double num = 0.0, den = 0.0;
                    for (int q = 0; q < np; ++q) {
                        double D = weights ? (double)weights[prov[q]] : 1.0;
                        num += D * load_x(in, elem, (size_t)prov[q] * (size_t)P + (size_t)p);
                        den += D;
                    }
                    ((double *)out)[o] = num / den;
                } else {
                    /* the fixed-order binary32 form, as in oracle_segment_aggregate_ordered_f32 */
                    float acc = 0.0f;
                    for (int q = 0; q < np; ++q) {
                        size_t off = (size_t)prov[q] * (size_t)P + (size_t)p;
                        float x = (elem == 4) ? ((const float *)in)[off] : bf16_to_f32(((const uint16_t *)in)[off]);
                        float D = weights ? weights[prov[q]] : 1.0f;
                        if (q == 0) { volatile float prod = D * x; acc = (np == 1) ? x : prod; }
                        else acc = fmaf(D, x, acc);
                    }
                    if (np > 1) { volatile float qq = acc * rden32; acc = qq; }
                    if (elem == 4) ((float *)out)[o] = acc;
                    else ((uint16_t *)out)[o] = oracle_f32_to_bf16_rne(acc);
                }
            }
        }
    }
    free(prov);
    return 0;
}
