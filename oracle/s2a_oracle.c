/*
 * CPU fp64 oracle for shifted sparse attention (S2-Attn), forward and backward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * operator computes; it exists so that tests and the benchmark's CPU-baseline
 * leg can check and time it.  The GPU library never calls it and shares no code
 * with it.
 *
 * What it computes (Algorithm 1 and Section 3.2 of the LongLoRA paper; Eq. 1 for
 * the attention itself), written in index form rather than with materialised
 * rolls:
 *
 *   - the N tokens are split into N/G groups of G consecutive tokens;
 *   - in the second half of the heads (h >= H/2) the tokens are first rolled by
 *     -G/2, i.e. rolled position p holds original token (p + G/2) mod N, so the
 *     group boundaries sit half a group later and the last group wraps (it
 *     holds the last G/2 and the first G/2 tokens);
 *   - softmax attention (Eq. 1, with the usual `scale` on the scores) runs
 *     inside each group, causally in rolled order;
 *   - the second half of the heads is rolled back by +G/2, so outputs are
 *     indexed by original token.
 *
 * For original token t of head h with shift s_h (0 or G/2):
 *     p      = (t - s_h) mod N            rolled position
 *     g      = floor(p / G)               its group
 *     A(t,h) = { t' = (p' + s_h) mod N : g*G <= p' <= p }    attended keys
 * With kv = floor(h / (H/Hkv)) (grouped-query head mapping; the paper's
 * Algorithm 1 has H == Hkv):
 *     z_{t'}      = scale * sum_c q[b,t,h,c] * k[b,t',kv,c]
 *     lse[b,h,t]  = log sum_{t' in A} exp(z_{t'})
 *     o[b,t,h,:]  = sum_{t' in A} exp(z_{t'} - lse) * v[b,t',kv,:]
 *
 * Backward (the gradient of the above; the paper trains through it by
 * autograd), with P_{t t'} = exp(z_{t'} - lse_t) on A and D_t = dO_t . o_t:
 *     dS_{t t'}       = P_{t t'} * (dO[b,t,h,:] . v[b,t',kv,:] - D_t)
 *     dQ[b,t,h,:]     = scale * sum_{t' in A(t,h)} dS_{t t'} * k[b,t',kv,:]
 *     dK[b,t',kv,:]   = scale * sum_{h in kv} sum_{t : t' in A(t,h)} dS_{t t'} * q[b,t,h,:]
 *     dV[b,t',kv,:]   = sum_{h in kv} sum_{t : t' in A(t,h)} P_{t t'} * dO[b,t,h,:]
 *
 * Every output row is computed on its own, straight from these sums: no tiling,
 * no online softmax, no reordering.  Inputs are either fp64 arrays or bf16 bit
 * patterns (widened exactly to fp64); all arithmetic is fp64.
 *
 * Parity pins (tests/test_oracle_*.py): the paper's worked example of group
 * membership, an independent transcription of Algorithm 1 with autograd,
 * brute-force loops on tiny inputs, closed forms, finite differences,
 * dependency structure, the GQA->MHA reduction and the paper's FLOP table.
 * The absolute values of o, dq, dk, dv on the benchmark configurations are not
 * printed anywhere in the paper: for those, parity is pinned only through
 * these properties of the oracle that produces them.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define S2A_ORACLE_F64 0
#define S2A_ORACLE_BF16 1

typedef struct {
    int B, N, H, Hkv, d, G;
    int n_unshifted; /* heads [0, n_unshifted) use shift 0, the rest use `shift` */
    int shift;       /* G/2 in the paper; sign = roll direction                 */
    int dtype;
    double scale;
    int variant;     /* 0 = Algorithm 1; 1 = variant 2 of Appendix B; 2 = variant 3 of Appendix B */
} s2a_dims;

static double bf16_to_f64(uint16_t bits) {
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Copy one length-d row, starting at element `off`, into fp64. */
static void load_row(const void* base, size_t off, int d, int dtype, double* dst) {
    if (dtype == S2A_ORACLE_F64) {
        const double* p = (const double*)base + off;
        for (int c = 0; c < d; ++c) dst[c] = p[c];
    } else {
        const uint16_t* p = (const uint16_t*)base + off;
        for (int c = 0; c < d; ++c) dst[c] = bf16_to_f64(p[c]);
    }
}

static int mod_n(long long x, int n) {
    long long r = x % n;
    return (int)(r < 0 ? r + n : r);
}

/* shift of head h (Section 3.2: half of the heads use the shifted partition) */
static int head_shift(const s2a_dims* D, int h) { return h < D->n_unshifted ? 0 : D->shift; }

/*
 * Variants 2 and 3 of Appendix B concern the one group of a shifted head that wraps around the
 * sequence end: it holds the last tokens of the sequence ("tail") followed by the first ones
 * ("front"), so that in Algorithm 1 the front tokens attend the tail tokens.
 *   variant 2 (Appendix B, Table 8; separate groups for the shifted tokens): the group is cut in two at the wrap;
 *             front tokens attend front tokens only, tail tokens attend tail tokens only.
 *   variant 3 (Appendix B, Table 8; the front and the shifted tokens exchanged): the two parts change places, so
 *             the group is in original token order: front tokens come first (and attend only
 *             themselves), tail tokens follow and attend all front tokens and the tail tokens before
 *             them.
 * pw is the rolled position of original token 0; the group containing it is the wrapped one (unless
 * pw is a group boundary, where nothing wraps).
 */
static int wrap_pos(const s2a_dims* D, int s) { return mod_n(-(long long)s, D->N); }

/* up to two inclusive ranges of rolled positions, in the order in which the group is attended */
typedef struct {
    int n;
    int lo[2], hi[2];
} s2a_ranges;

static int wrapped_at(const s2a_dims* D, int s, int g_first) {
    if (s == 0) return -1;
    const int pw = wrap_pos(D, s);
    return (pw > g_first && pw < g_first + D->G) ? pw : -1;
}

/* keys attended by the query at rolled position p (head with shift s) */
static s2a_ranges keys_of_query(const s2a_dims* D, int s, int p) {
    s2a_ranges r;
    const int g_first = (p / D->G) * D->G;
    const int pw = D->variant ? wrapped_at(D, s, g_first) : -1;
    r.n = 1, r.lo[0] = g_first, r.hi[0] = p;
    if (pw >= 0) {
        if (p >= pw) {
            r.lo[0] = pw; /* a front token: front tokens up to itself, in both variants */
        } else if (D->variant == 2) {
            r.n = 2; /* a tail token after the swap: every front token, then the tail up to itself */
            r.lo[0] = pw, r.hi[0] = g_first + D->G - 1;
            r.lo[1] = g_first, r.hi[1] = p;
        }
    }
    return r;
}

/* queries that attend the key at rolled position pk */
static s2a_ranges queries_of_key(const s2a_dims* D, int s, int pk) {
    s2a_ranges r;
    const int g_first = (pk / D->G) * D->G;
    const int g_last = g_first + D->G - 1;
    const int pw = D->variant ? wrapped_at(D, s, g_first) : -1;
    r.n = 1, r.lo[0] = pk, r.hi[0] = g_last;
    if (pw >= 0) {
        if (pk < pw) {
            r.hi[0] = pw - 1; /* a tail key: the tail tokens from itself on, in both variants */
        } else if (D->variant == 2) {
            r.n = 2; /* a front key after the swap: the front tokens from itself on, then every tail token */
            r.lo[1] = g_first, r.hi[1] = pw - 1;
        }
    }
    return r;
}

static size_t q_off(const s2a_dims* D, int b, int t, int h) {
    return (((size_t)b * D->N + t) * D->H + h) * (size_t)D->d;
}
static size_t kv_off(const s2a_dims* D, int b, int t, int hk) {
    return (((size_t)b * D->N + t) * D->Hkv + hk) * (size_t)D->d;
}

static double dot(const double* a, const double* b, int d) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += a[c] * b[c];
    return s;
}

/*
 * Forward for one (b, h, t) row.  zbuf has room for G scores, krow for d values.
 * Returns lse; writes o_row (d values) if o_row != NULL.
 */
static double fwd_row(const s2a_dims* D, const void* q, const void* k, const void* v, int b, int h, int t,
                      double* qrow, double* krow, double* zbuf, double* o_row) {
    const int s = head_shift(D, h);
    const int hk = h / (D->H / D->Hkv);
    const int p = mod_n((long long)t - s, D->N);
    const s2a_ranges att = keys_of_query(D, s, p);
    int n_att = 0;

    load_row(q, q_off(D, b, t, h), D->d, D->dtype, qrow);
    double zmax = -INFINITY;
    for (int a = 0; a < att.n; ++a) {
        for (int pp = att.lo[a]; pp <= att.hi[a]; ++pp, ++n_att) {
            const int tk = mod_n((long long)pp + s, D->N);
            load_row(k, kv_off(D, b, tk, hk), D->d, D->dtype, krow);
            zbuf[n_att] = D->scale * dot(qrow, krow, D->d);
            if (zbuf[n_att] > zmax) zmax = zbuf[n_att];
        }
    }
    double sum = 0.0;
    for (int i = 0; i < n_att; ++i) sum += exp(zbuf[i] - zmax);
    const double lse = zmax + log(sum);
    if (o_row) {
        for (int c = 0; c < D->d; ++c) o_row[c] = 0.0;
        int i = 0;
        for (int a = 0; a < att.n; ++a) {
            for (int pp = att.lo[a]; pp <= att.hi[a]; ++pp, ++i) {
                const int tk = mod_n((long long)pp + s, D->N);
                const double w = exp(zbuf[i] - lse);
                load_row(v, kv_off(D, b, tk, hk), D->d, D->dtype, krow);
                for (int c = 0; c < D->d; ++c) o_row[c] += w * krow[c];
            }
        }
    }
    return lse;
}

static int check_dims(const s2a_dims* D) {
    if (D->B <= 0 || D->N <= 0 || D->H <= 0 || D->Hkv <= 0 || D->d <= 0 || D->G <= 0) return -1;
    if (D->N % D->G) return -1;
    if (D->H % D->Hkv) return -1;
    if (D->n_unshifted < 0 || D->n_unshifted > D->H) return -1;
    if (D->dtype != S2A_ORACLE_F64 && D->dtype != S2A_ORACLE_BF16) return -1;
    return 0;
}

/*
 * Forward.  rows == NULL: every (b,t,h); o is [B,N,H,d], lse is [B,H,N].
 * rows != NULL: n_rows triples (b,h,t); o is [n_rows,d], lse is [n_rows].
 */
int s2a_oracle_fwd_ex(const void* q, const void* k, const void* v, int dtype, int B, int N, int H, int Hkv, int d,
                      int G, double scale, int n_unshifted, int shift, int variant, const int* rows,
                      long long n_rows, double* o, double* lse) {
    s2a_dims D = {B, N, H, Hkv, d, G, n_unshifted, shift, dtype, scale, variant};
    if (check_dims(&D)) return -1;
    const long long total = rows ? n_rows : (long long)B * H * N;
    int err = 0;
#pragma omp parallel
    {
        double* qrow = (double*)malloc(sizeof(double) * (size_t)d);
        double* krow = (double*)malloc(sizeof(double) * (size_t)d);
        double* zbuf = (double*)malloc(sizeof(double) * (size_t)G);
        if (!qrow || !krow || !zbuf) {
#pragma omp atomic write
            err = 1;
        } else {
#pragma omp for schedule(dynamic, 16)
            for (long long r = 0; r < total; ++r) {
                int b, h, t;
                if (rows) {
                    b = rows[3 * r], h = rows[3 * r + 1], t = rows[3 * r + 2];
                } else {
                    b = (int)(r / ((long long)H * N));
                    h = (int)((r / N) % H);
                    t = (int)(r % N);
                }
                double* o_row = rows ? o + (size_t)r * d : o + q_off(&D, b, t, h);
                double l = fwd_row(&D, q, k, v, b, h, t, qrow, krow, zbuf, o_row);
                if (rows) lse[r] = l;
                else lse[((size_t)b * H + h) * N + t] = l;
            }
        }
        free(qrow), free(krow), free(zbuf);
    }
    return err ? -2 : 0;
}

/* Paper defaults: second half of the heads shifted by G/2 (Algorithm 1). */
int s2a_oracle_fwd(const void* q, const void* k, const void* v, int dtype, int B, int N, int H, int Hkv, int d,
                   int G, double scale, const int* rows, long long n_rows, double* o, double* lse) {
    if ((G & 1) || (H & 1)) return -1;
    return s2a_oracle_fwd_ex(q, k, v, dtype, B, N, H, Hkv, d, G, scale, H / 2, G / 2, 0, rows, n_rows, o, lse);
}

/*
 * Backward.
 *   q_rows  : n_q triples (b,h,t)   -> dq [n_q, d]      (NULL: all, dq is [B,N,H,d])
 *   kv_rows : n_kv triples (b,hk,t) -> dk, dv [n_kv, d] (NULL: all, [B,N,Hkv,d])
 * Pass n_q = 0 with a non-NULL q_rows (or n_kv = 0 likewise) to skip that part.
 * The statistics lse_t and D_t of every query row that is needed are computed
 * first (a forward pass over those rows), then every requested gradient row is
 * summed on its own from the definition.
 */
int s2a_oracle_bwd_ex(const void* q, const void* k, const void* v, const void* dO, int dtype, int B, int N, int H,
                      int Hkv, int d, int G, double scale, int n_unshifted, int shift, int variant,
                      const int* q_rows, long long n_q, const int* kv_rows, long long n_kv, double* dq, double* dk,
                      double* dv) {
    s2a_dims D = {B, N, H, Hkv, d, G, n_unshifted, shift, dtype, scale, variant};
    if (check_dims(&D)) return -1;
    const int r = H / Hkv;
    const size_t n_stat = (size_t)B * H * N;
    unsigned char* need = (unsigned char*)calloc(n_stat, 1);
    double* lse = (double*)malloc(sizeof(double) * n_stat);
    double* Dsum = (double*)malloc(sizeof(double) * n_stat);
    if (!need || !lse || !Dsum) {
        free(need), free(lse), free(Dsum);
        return -2;
    }
    const long long tot_q = q_rows ? n_q : (long long)B * H * N;
    const long long tot_kv = kv_rows ? n_kv : (long long)B * Hkv * N;

    /* which query rows' statistics are needed */
    if (!q_rows) {
        memset(need, 1, n_stat);
    } else {
        for (long long i = 0; i < n_q; ++i)
            need[((size_t)q_rows[3 * i] * H + q_rows[3 * i + 1]) * N + q_rows[3 * i + 2]] = 1;
    }
    if (!kv_rows) {
        memset(need, 1, n_stat);
    } else {
        for (long long i = 0; i < n_kv; ++i) {
            const int b = kv_rows[3 * i], hk = kv_rows[3 * i + 1], tk = kv_rows[3 * i + 2];
            for (int h = hk * r; h < (hk + 1) * r; ++h) {
                const int s = head_shift(&D, h);
                const int pk = mod_n((long long)tk - s, N);
                const s2a_ranges qs = queries_of_key(&D, s, pk); /* the queries that attend tk */
                for (int a = 0; a < qs.n; ++a)
                    for (int p = qs.lo[a]; p <= qs.hi[a]; ++p) need[((size_t)b * H + h) * N + mod_n((long long)p + s, N)] = 1;
            }
        }
    }

    int err = 0;
#pragma omp parallel
    {
        double* qrow = (double*)malloc(sizeof(double) * (size_t)d);
        double* krow = (double*)malloc(sizeof(double) * (size_t)d);
        double* vrow = (double*)malloc(sizeof(double) * (size_t)d);
        double* dorow = (double*)malloc(sizeof(double) * (size_t)d);
        double* orow = (double*)malloc(sizeof(double) * (size_t)d);
        double* zbuf = (double*)malloc(sizeof(double) * (size_t)G);
        if (!qrow || !krow || !vrow || !dorow || !orow || !zbuf) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
            /* pass 1: lse_t and D_t = dO_t . o_t */
#pragma omp for schedule(dynamic, 16)
            for (long long idx = 0; idx < (long long)n_stat; ++idx) {
                if (!need[idx]) continue;
                const int b = (int)(idx / ((long long)H * N));
                const int h = (int)((idx / N) % H);
                const int t = (int)(idx % N);
                lse[idx] = fwd_row(&D, q, k, v, b, h, t, qrow, krow, zbuf, orow);
                load_row(dO, q_off(&D, b, t, h), d, dtype, dorow);
                Dsum[idx] = dot(dorow, orow, d);
            }

            /* pass 2a: dQ rows */
#pragma omp for schedule(dynamic, 16)
            for (long long i = 0; i < tot_q; ++i) {
                int b, h, t;
                if (q_rows) {
                    b = q_rows[3 * i], h = q_rows[3 * i + 1], t = q_rows[3 * i + 2];
                } else {
                    b = (int)(i / ((long long)H * N));
                    h = (int)((i / N) % H);
                    t = (int)(i % N);
                }
                const size_t si = ((size_t)b * H + h) * N + t;
                const int s = head_shift(&D, h);
                const int hk = h / r;
                const int p = mod_n((long long)t - s, N);
                const s2a_ranges att = keys_of_query(&D, s, p);
                double* out = q_rows ? dq + (size_t)i * d : dq + q_off(&D, b, t, h);
                for (int c = 0; c < d; ++c) out[c] = 0.0;
                load_row(q, q_off(&D, b, t, h), d, dtype, qrow);
                load_row(dO, q_off(&D, b, t, h), d, dtype, dorow);
                for (int a = 0; a < att.n; ++a) {
                    for (int pp = att.lo[a]; pp <= att.hi[a]; ++pp) {
                        const int tk = mod_n((long long)pp + s, N);
                        load_row(k, kv_off(&D, b, tk, hk), d, dtype, krow);
                        load_row(v, kv_off(&D, b, tk, hk), d, dtype, vrow);
                        const double P = exp(scale * dot(qrow, krow, d) - lse[si]);
                        const double dS = P * (dot(dorow, vrow, d) - Dsum[si]);
                        for (int c = 0; c < d; ++c) out[c] += scale * dS * krow[c];
                    }
                }
            }

            /* pass 2b: dK and dV rows */
#pragma omp for schedule(dynamic, 4)
            for (long long i = 0; i < tot_kv; ++i) {
                int b, hk, tk;
                if (kv_rows) {
                    b = kv_rows[3 * i], hk = kv_rows[3 * i + 1], tk = kv_rows[3 * i + 2];
                } else {
                    b = (int)(i / ((long long)Hkv * N));
                    hk = (int)((i / N) % Hkv);
                    tk = (int)(i % N);
                }
                double* out_k = kv_rows ? dk + (size_t)i * d : dk + kv_off(&D, b, tk, hk);
                double* out_v = kv_rows ? dv + (size_t)i * d : dv + kv_off(&D, b, tk, hk);
                for (int c = 0; c < d; ++c) out_k[c] = 0.0, out_v[c] = 0.0;
                load_row(k, kv_off(&D, b, tk, hk), d, dtype, krow);
                load_row(v, kv_off(&D, b, tk, hk), d, dtype, vrow);
                for (int h = hk * r; h < (hk + 1) * r; ++h) {
                    const int s = head_shift(&D, h);
                    const int pk = mod_n((long long)tk - s, N);
                    const s2a_ranges qs = queries_of_key(&D, s, pk);
                    for (int a = 0; a < qs.n; ++a) {
                        for (int p = qs.lo[a]; p <= qs.hi[a]; ++p) {
                            const int t = mod_n((long long)p + s, N);
                            const size_t si = ((size_t)b * H + h) * N + t;
                            load_row(q, q_off(&D, b, t, h), d, dtype, qrow);
                            load_row(dO, q_off(&D, b, t, h), d, dtype, dorow);
                            const double P = exp(scale * dot(qrow, krow, d) - lse[si]);
                            const double dS = P * (dot(dorow, vrow, d) - Dsum[si]);
                            for (int c = 0; c < d; ++c) {
                                out_v[c] += P * dorow[c];
                                out_k[c] += scale * dS * qrow[c];
                            }
                        }
                    }
                }
            }
        }
        free(qrow), free(krow), free(vrow), free(dorow), free(orow), free(zbuf);
    }
    free(need), free(lse), free(Dsum);
    return err ? -2 : 0;
}

int s2a_oracle_bwd(const void* q, const void* k, const void* v, const void* dO, int dtype, int B, int N, int H,
                   int Hkv, int d, int G, double scale, const int* q_rows, long long n_q, const int* kv_rows,
                   long long n_kv, double* dq, double* dk, double* dv) {
    if ((G & 1) || (H & 1)) return -1;
    return s2a_oracle_bwd_ex(q, k, v, dO, dtype, B, N, H, Hkv, d, G, scale, H / 2, G / 2, 0, q_rows, n_q, kv_rows,
                             n_kv, dq, dk, dv);
}

/*
 * Group membership alone (for pinning against the paper's worked example):
 * writes the original-token ids attended by (h, t), in rolled order, into `out`
 * (room for G ints) and returns their count.
 */
int s2a_oracle_attended(int N, int H, int G, int h, int t, int* out) {
    if (N <= 0 || G <= 0 || N % G || (G & 1) || (H & 1) || h < 0 || h >= H || t < 0 || t >= N) return -1;
    const int s = h < H / 2 ? 0 : G / 2;
    const int p = mod_n((long long)t - s, N);
    const int p_first = (p / G) * G;
    int n = 0;
    for (int pp = p_first; pp <= p; ++pp) out[n++] = mod_n((long long)pp + s, N);
    return n;
}

int s2a_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
