/*
 * usv_oracle.c -- plain fp64 CPU statement of the USV sparsified-attention path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct checker
 * that the CUDA library is compared against.  It shares no code, header,
 * table or helper with the CUDA path, and the product never calls it: only the
 * test-suite, the smoke check and the benchmark's cpu-baseline leg do.
 *
 * Everything is evaluated in double precision on the exact values of the bf16
 * inputs.  Loops are written in the order of the paper's definitions; the only
 * parallelism is an OpenMP "for" over independent outer items.
 *
 * What follows which passage (equations numbered in order of appearance):
 *   usvo_dense_masked_attn  Sec. 3.2, Eq. 5: softmax((QK^T + log M)/sqrt(d_k)) V with the
 *                           block-structured mask M written out as an N x N matrix.
 *   usvo_sparse_attn        the same Eq. 5 evaluated only over the columns where M = 1
 *                           (mathematically identical; used where N x N is too large).
 *   usvo_block_pool /       coarse stage of "top-k cube selection" (Fig. 2 caption, Sec. 2.2):
 *   usvo_block_scores /     the paper names the step but prints no score function; the
 *   usvo_select_blocks      reading used here is mean-pooled block queries/keys, scaled dot
 *                           product, k largest per row, ties to the lowest block index.
 *                           PARITY UNPINNED by the paper for the choice of score function
 *                           (pinned only for the top-k rule itself, by brute force).
 *   usvo_merge_descriptors  Sec. 3.3, Eq. 7 (head-averaged key descriptor) and the
 *                           normalisation inside Eq. 8.
 *   usvo_merge_match        Sec. 3.3, Eq. 6 (one destination per (s_t,s_h,s_w) block; reading:
 *                           the block's first token), Eq. 8 (cosine), Eq. 9 (arg-max over all
 *                           destinations of the same batch element, ties to the lowest index).
 *   usvo_merge_select       Sec. 3.3, Eq. 10-11: the r sources with largest u, ties to the
 *                           lowest source index.
 *   usvo_merge_positions    Sec. 3.3, Eq. 14: merged order [U ascending || B ascending].
 *   usvo_merge_apply        Sec. 3.3, Eq. 12-13: mean aggregation into destinations.
 *   usvo_unmerge            Sec. 3.3, Eq. 15: copy back by stored plan.
 *   usvo_key_marginal       Sec. 3.4, Eq. 16: attention weights (here: of the block-masked
 *                           attention of Eq. 5) averaged over heads and queries.
 *   usvo_entropy            Sec. 3.4, Eq. 17: entropy of that marginal, normalised by log N.
 *   usvo_allocate           Sec. 3.4, Eq. 18-19: w = (1-h)^gamma, rho_l = clip(rho_bar w_l / mean w).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define USVO_BS 64 /* tokens per attention block (the workload definition fixes 64) */

/* ---------------------------------------------------------------- bf16 <-> double */

static double bf16_val(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* Round a double straight to bf16 (8-bit significand), nearest-even, no float detour. */
uint16_t usvo_double_to_bf16(double x) {
    if (x != x) return 0x7fc0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7f80;
    int e;
    double m = frexp(a, &e); /* a = m * 2^e, m in [0.5,1) */
    double q;                /* quantum of the target grid at this magnitude */
    if (e - 8 < -133) q = ldexp(1.0, -133); /* bf16 subnormal spacing */
    else q = ldexp(1.0, e - 8);
    (void)m;
    double r = nearbyint(a / q) * q; /* default rounding mode = nearest-even */
    float f = (float)r;              /* exact: r has at most 8 significant bits */
    if (isinf(f)) return sign | 0x7f80;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u >> 16) >= 0x7f80) return sign | 0x7f80;
    return sign | (uint16_t)(u >> 16);
}

void usvo_round_to_bf16(const double* x, int64_t n, uint16_t* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = usvo_double_to_bf16(x[i]);
}

void usvo_bf16_to_double(const uint16_t* x, int64_t n, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_val(x[i]);
}

int usvo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- coarse stage */

/* Mean of the valid tokens (index < N) of every 64-token block.
 * x: bf16 [B,H,*,d] with element strides (sb,sh,sn), d contiguous.  out: [B,H,NB,d]. */
void usvo_block_pool(const uint16_t* x, int B, int H, int N, int d, int64_t sb, int64_t sh,
                     int64_t sn, double* out) {
    int NB = (N + USVO_BS - 1) / USVO_BS;
#pragma omp parallel for collapse(2) schedule(static)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int I = 0; I < NB; ++I) {
            int b = bh / H, h = bh % H;
            int lo = I * USVO_BS;
            int hi = lo + USVO_BS < N ? lo + USVO_BS : N;
            double* o = out + ((int64_t)bh * NB + I) * d;
            for (int e = 0; e < d; ++e) {
                double s = 0.0;
                for (int n = lo; n < hi; ++n) s += bf16_val(x[b * sb + h * sh + n * sn + e]);
                o[e] = s / (double)(hi - lo);
            }
        }
    }
}

/* S[b,h,I,J] = <qbar_I, kbar_J> / sqrt(d). */
void usvo_block_scores(const double* qbar, const double* kbar, int B, int H, int NBq, int NBk,
                       int d, double* s) {
    double inv = 1.0 / sqrt((double)d);
#pragma omp parallel for collapse(2) schedule(static)
    for (int bh = 0; bh < B * H; ++bh) {
        for (int I = 0; I < NBq; ++I) {
            const double* q = qbar + ((int64_t)bh * NBq + I) * d;
            for (int J = 0; J < NBk; ++J) {
                const double* k = kbar + ((int64_t)bh * NBk + J) * d;
                double acc = 0.0;
                for (int e = 0; e < d; ++e) acc += q[e] * k[e];
                s[((int64_t)bh * NBq + I) * NBk + J] = acc * inv;
            }
        }
    }
}

typedef struct {
    double key; /* value to sort descending */
    int idx;    /* tie-break ascending */
} usvo_pair;

static int cmp_desc_then_idx(const void* a, const void* b) {
    const usvo_pair* x = (const usvo_pair*)a;
    const usvo_pair* y = (const usvo_pair*)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

static int cmp_int(const void* a, const void* b) {
    int x = *(const int*)a, y = *(const int*)b;
    return (x > y) - (x < y);
}

/* For each (b,h,I): order J by (score descending, J ascending), keep the first k_h, emit them
 * in ascending J; tail of the kmax-wide row is -1.
 * gap[b,h,I] = (s_(k) - s_(k+1)) / max(|s_(k)|,|s_(k+1)|,1e-30), or +inf when k_h == NBk. */
void usvo_select_blocks(const double* s, int B, int H, int NBq, int NBk, const int32_t* k_per_head,
                        int kmax, int32_t* sel, double* gap) {
#pragma omp parallel
    {
        usvo_pair* p = (usvo_pair*)malloc(sizeof(usvo_pair) * (size_t)NBk);
#pragma omp for collapse(2) schedule(static)
        for (int bh = 0; bh < B * H; ++bh) {
            for (int I = 0; I < NBq; ++I) {
                int h = bh % H;
                int k = k_per_head[h];
                const double* row = s + ((int64_t)bh * NBq + I) * NBk;
                for (int J = 0; J < NBk; ++J) {
                    p[J].key = row[J];
                    p[J].idx = J;
                }
                qsort(p, (size_t)NBk, sizeof(usvo_pair), cmp_desc_then_idx);
                int32_t* out = sel + ((int64_t)bh * NBq + I) * kmax;
                for (int t = 0; t < k; ++t) out[t] = p[t].idx;
                qsort(out, (size_t)k, sizeof(int32_t), cmp_int);
                for (int t = k; t < kmax; ++t) out[t] = -1;
                if (gap) {
                    double g = INFINITY;
                    if (k < NBk) {
                        double a = p[k - 1].key, c = p[k].key;
                        double den = fmax(fmax(fabs(a), fabs(c)), 1e-30);
                        g = (a - c) / den;
                    }
                    gap[(int64_t)bh * NBq + I] = g;
                }
            }
        }
        free(p);
    }
}

/* ---------------------------------------------------------------- attention */

/* Literal Eq. 5 on one (b,h): builds the N x N mask from the block selection, adds log M to
 * the logits, applies the scale, softmax over all N columns, multiplies by V.
 * Only for small N (memory N*N doubles per thread).
 * q,k,v: bf16 with strides; sel: [B,H,NB,kmax]; o: [B,H,N,d]; prob_rowsum (optional): [B,H,N]
 * receives the sum of each softmax row (should be 1). */
void usvo_dense_masked_attn(const uint16_t* q, const uint16_t* k, const uint16_t* v, int B, int H,
                            int N, int d, int64_t sb, int64_t sh, int64_t sn, const int32_t* sel,
                            const int32_t* k_per_head, int kmax, double scale, double* o,
                            double* prob_rowsum) {
    int NB = (N + USVO_BS - 1) / USVO_BS;
#pragma omp parallel for schedule(dynamic)
    for (int bh = 0; bh < B * H; ++bh) {
        int b = bh / H, h = bh % H;
        int64_t base = b * sb + h * sh;
        double* M = (double*)malloc(sizeof(double) * (size_t)N * N);
        double* A = (double*)malloc(sizeof(double) * (size_t)N * N);
        for (int i = 0; i < N; ++i) {
            int I = i / USVO_BS;
            const int32_t* row = sel + ((int64_t)bh * NB + I) * kmax;
            for (int j = 0; j < N; ++j) M[(size_t)i * N + j] = 0.0;
            for (int t = 0; t < k_per_head[h]; ++t) {
                int J = row[t];
                if (J < 0) continue;
                for (int j = J * USVO_BS; j < (J + 1) * USVO_BS && j < N; ++j)
                    M[(size_t)i * N + j] = 1.0;
            }
        }
        for (int i = 0; i < N; ++i) {
            for (int j = 0; j < N; ++j) {
                double acc = 0.0;
                for (int e = 0; e < d; ++e)
                    acc += bf16_val(q[base + i * sn + e]) * bf16_val(k[base + j * sn + e]);
                A[(size_t)i * N + j] = (acc + log(M[(size_t)i * N + j])) * scale; /* log 0 = -inf */
            }
        }
        for (int i = 0; i < N; ++i) {
            double* a = A + (size_t)i * N;
            double mx = -INFINITY;
            for (int j = 0; j < N; ++j) mx = a[j] > mx ? a[j] : mx;
            double sum = 0.0;
            for (int j = 0; j < N; ++j) {
                a[j] = exp(a[j] - mx);
                sum += a[j];
            }
            double rs = 0.0;
            for (int j = 0; j < N; ++j) {
                a[j] /= sum;
                rs += a[j];
            }
            if (prob_rowsum) prob_rowsum[(int64_t)bh * N + i] = rs;
            double* out = o + ((int64_t)bh * N + i) * d;
            for (int e = 0; e < d; ++e) {
                double acc = 0.0;
                for (int j = 0; j < N; ++j) acc += a[j] * bf16_val(v[base + j * sn + e]);
                out[e] = acc;
            }
        }
        free(M);
        free(A);
    }
}

/* Eq. 5 restricted to the allowed columns, for a list of query blocks.
 * qb_list: n_qb triples (b,h,I).  o: [n_qb,64,d]; lse: [n_qb,64] (natural log of the softmax
 * denominator including the max).  Rows with token index >= N are written as 0 (lse = 0).
 * q/k/v each have their own strides: sq[3], sk[3], sv[3] = (sb,sh,sn). */
void usvo_sparse_attn(const uint16_t* q, const int64_t* sq, const uint16_t* k, const int64_t* sk,
                      const uint16_t* v, const int64_t* sv, int B, int H, int N, int d,
                      const int32_t* sel, const int32_t* k_per_head, int kmax, double scale,
                      const int32_t* qb_list, int n_qb, double* o, double* lse) {
    (void)B;
    int NB = (N + USVO_BS - 1) / USVO_BS;
#pragma omp parallel
    {
        size_t cap = (size_t)kmax * USVO_BS;
        double* Kd = (double*)malloc(sizeof(double) * cap * d);
        double* Vd = (double*)malloc(sizeof(double) * cap * d);
        double* a = (double*)malloc(sizeof(double) * cap);
        double* qd = (double*)malloc(sizeof(double) * d);
#pragma omp for schedule(dynamic)
        for (int w = 0; w < n_qb; ++w) {
            int b = qb_list[3 * w], h = qb_list[3 * w + 1], I = qb_list[3 * w + 2];
            const int32_t* row = sel + (((int64_t)b * H + h) * NB + I) * kmax;
            /* gather the allowed, valid key/value rows */
            int nk = 0;
            for (int t = 0; t < k_per_head[h]; ++t) {
                int J = row[t];
                if (J < 0) continue;
                for (int j = J * USVO_BS; j < (J + 1) * USVO_BS && j < N; ++j) {
                    for (int e = 0; e < d; ++e) {
                        Kd[(size_t)nk * d + e] = bf16_val(k[b * sk[0] + h * sk[1] + j * sk[2] + e]);
                        Vd[(size_t)nk * d + e] = bf16_val(v[b * sv[0] + h * sv[1] + j * sv[2] + e]);
                    }
                    ++nk;
                }
            }
            for (int r = 0; r < USVO_BS; ++r) {
                int i = I * USVO_BS + r;
                double* out = o + ((int64_t)w * USVO_BS + r) * d;
                if (i >= N || nk == 0) {
                    for (int e = 0; e < d; ++e) out[e] = 0.0;
                    if (lse) lse[(int64_t)w * USVO_BS + r] = 0.0;
                    continue;
                }
                for (int e = 0; e < d; ++e) qd[e] = bf16_val(q[b * sq[0] + h * sq[1] + i * sq[2] + e]);
                double mx = -INFINITY;
                for (int j = 0; j < nk; ++j) {
                    double acc = 0.0;
                    const double* kr = Kd + (size_t)j * d;
                    for (int e = 0; e < d; ++e) acc += qd[e] * kr[e];
                    a[j] = acc * scale;
                    mx = a[j] > mx ? a[j] : mx;
                }
                double sum = 0.0;
                for (int j = 0; j < nk; ++j) {
                    a[j] = exp(a[j] - mx);
                    sum += a[j];
                }
                for (int e = 0; e < d; ++e) out[e] = 0.0;
                for (int j = 0; j < nk; ++j) {
                    double p = a[j] / sum;
                    const double* vr = Vd + (size_t)j * d;
                    for (int e = 0; e < d; ++e) out[e] += p * vr[e];
                }
                if (lse) lse[(int64_t)w * USVO_BS + r] = mx + log(sum);
            }
        }
        free(Kd);
        free(Vd);
        free(a);
        free(qd);
    }
}

/* ---------------------------------------------------------------- token merging */

/* Eq. 6: the destination of each (st,sh,sw) block is its first token in raster order. */
static int is_destination(int n, int Hh, int W, int st, int shh, int sw) {
    int x = n % W;
    int y = (n / W) % Hh;
    int t = n / (W * Hh);
    return (t % st == 0) && (y % shh == 0) && (x % sw == 0);
}

void usvo_destination_mask(int T, int Hh, int W, int st, int shh, int sw, uint8_t* is_dst) {
    int N = T * Hh * W;
    for (int n = 0; n < N; ++n) is_dst[n] = (uint8_t)is_destination(n, Hh, W, st, shh, sw);
}

/* Eq. 7 then the unit-normalisation of Eq. 8.  metric: bf16 [B,N,Hm,dm] contiguous.
 * mhat: [B,N,dm].  A zero descriptor stays zero (norm clamped at 1e-12). */
void usvo_merge_descriptors(const uint16_t* metric, int B, int N, int Hm, int dm, double* mhat) {
#pragma omp parallel for schedule(static)
    for (int64_t bn = 0; bn < (int64_t)B * N; ++bn) {
        const uint16_t* src = metric + bn * Hm * dm;
        double* m = mhat + bn * dm;
        double nrm2 = 0.0;
        for (int e = 0; e < dm; ++e) {
            double s = 0.0;
            for (int h = 0; h < Hm; ++h) s += bf16_val(src[h * dm + e]);
            m[e] = s / (double)Hm;
            nrm2 += m[e] * m[e];
        }
        double nrm = sqrt(nrm2);
        if (nrm < 1e-12) nrm = 1e-12;
        for (int e = 0; e < dm; ++e) m[e] /= nrm;
    }
}

/* Eq. 8-9 for the sources listed in src_list (n_src pairs (b,i); i must be a source).
 * jstar[w] = lowest-index arg-max destination, u[w] = that cosine, u2[w] = the second largest
 * cosine over destinations (-inf if there is one destination only). */
void usvo_merge_match(const double* mhat, int B, int N, int dm, int T, int Hh, int W, int st,
                      int shh, int sw, const int32_t* src_list, int64_t n_src, int32_t* jstar,
                      double* u, double* u2) {
    (void)B;
    (void)T;
    int nd = 0;
    int32_t* dsts = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    for (int n = 0; n < N; ++n)
        if (is_destination(n, Hh, W, st, shh, sw)) dsts[nd++] = n;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t w = 0; w < n_src; ++w) {
        int b = src_list[2 * w], i = src_list[2 * w + 1];
        const double* mi = mhat + ((int64_t)b * N + i) * dm;
        double best = -INFINITY, second = -INFINITY;
        int bj = -1;
        for (int t = 0; t < nd; ++t) {
            int j = dsts[t];
            const double* mj = mhat + ((int64_t)b * N + j) * dm;
            double s = 0.0;
            for (int e = 0; e < dm; ++e) s += mi[e] * mj[e];
            if (s > best) { /* strict: an equal later j never replaces an earlier one */
                second = best;
                best = s;
                bj = j;
            } else if (s > second) {
                second = s;
            }
        }
        jstar[w] = bj;
        u[w] = best;
        u2[w] = second;
    }
    free(dsts);
}

/* Eq. 10-11 for one batch element: among the n_src sources (ascending indices src_idx, scores
 * u), mark the r with the largest u (ties to the lowest index).  merged[w] in {0,1}.
 * theta[0] = r-th largest u, theta[1] = (r+1)-th largest u (NaN where undefined). */
void usvo_merge_select(const int32_t* src_idx, const double* u, int n_src, int r, uint8_t* merged,
                       double* theta) {
    usvo_pair* p = (usvo_pair*)malloc(sizeof(usvo_pair) * (size_t)(n_src > 0 ? n_src : 1));
    for (int w = 0; w < n_src; ++w) {
        p[w].key = u[w];
        p[w].idx = w; /* src_idx ascending, so ordering by w == ordering by source index */
        merged[w] = 0;
    }
    (void)src_idx;
    qsort(p, (size_t)n_src, sizeof(usvo_pair), cmp_desc_then_idx);
    for (int t = 0; t < r; ++t) merged[p[t].idx] = 1;
    theta[0] = (r >= 1) ? p[r - 1].key : NAN;
    theta[1] = (r < n_src) ? p[r].key : NAN;
    free(p);
}

/* Eq. 14: position of every original token in the merged sequence [U asc || B asc].
 * dst_of[b,n] = j*(n) for merged sources, -1 otherwise.  pos[b,n] = row of the merged sequence
 * that token n reads back in Eq. 15.  Returns the merged length (same for all b) or -1 when
 * the batch elements disagree. */
int usvo_merge_positions(const int32_t* dst_of, int B, int T, int Hh, int W, int st, int shh,
                         int sw, int32_t* pos) {
    int N = T * Hh * W;
    int len0 = -1;
    for (int b = 0; b < B; ++b) {
        const int32_t* d = dst_of + (int64_t)b * N;
        int32_t* p = pos + (int64_t)b * N;
        int c = 0;
        for (int n = 0; n < N; ++n) /* U: sources that were not merged, ascending */
            if (!is_destination(n, Hh, W, st, shh, sw) && d[n] < 0) p[n] = c++;
        for (int n = 0; n < N; ++n) /* B: destinations, ascending */
            if (is_destination(n, Hh, W, st, shh, sw)) p[n] = c++;
        for (int n = 0; n < N; ++n) /* M: read back from the destination's row */
            if (!is_destination(n, Hh, W, st, shh, sw) && d[n] >= 0) p[n] = p[d[n]];
        if (len0 < 0) len0 = c;
        else if (len0 != c) return -1;
    }
    return len0;
}

/* Eq. 12-13: x bf16 [B,N,C]; out fp64 [B,Nm,C] with Nm = merged length. */
void usvo_merge_apply(const uint16_t* x, int B, int N, int C, const int32_t* dst_of,
                      const int32_t* pos, int Nm, double* out) {
    for (int b = 0; b < B; ++b) {
        const int32_t* d = dst_of + (int64_t)b * N;
        const int32_t* p = pos + (int64_t)b * N;
        double* ob = out + (int64_t)b * Nm * C;
        int32_t* cnt = (int32_t*)calloc((size_t)Nm, sizeof(int32_t));
        memset(ob, 0, sizeof(double) * (size_t)Nm * C);
        for (int n = 0; n < N; ++n) { /* every token adds itself to the row it maps to */
            int tgt = d[n] >= 0 ? d[n] : n; /* a merged source joins M(j*(n)); others stay */
            int row = p[tgt];
            cnt[row] += 1;
            const uint16_t* xr = x + ((int64_t)b * N + n) * C;
            double* orow = ob + (int64_t)row * C;
            for (int c = 0; c < C; ++c) orow[c] += bf16_val(xr[c]);
        }
#pragma omp parallel for schedule(static)
        for (int row = 0; row < Nm; ++row) {
            double* orow = ob + (int64_t)row * C;
            for (int c = 0; c < C; ++c) orow[c] /= (double)cnt[row];
        }
        free(cnt);
    }
}

/* Eq. 15: y bf16 [B,Nm,C] -> out bf16 [B,N,C] by pos. */
void usvo_unmerge(const uint16_t* y, int B, int N, int C, int Nm, const int32_t* pos,
                  uint16_t* out) {
#pragma omp parallel for schedule(static)
    for (int64_t bn = 0; bn < (int64_t)B * N; ++bn) {
        int b = (int)(bn / N);
        memcpy(out + bn * C, y + ((int64_t)b * Nm + pos[bn]) * C, sizeof(uint16_t) * (size_t)C);
    }
}

/* ---------------------------------------------------------------- entropy-aware scheduler */

/* Eq. 16: abar[b][j] = 1/(H N) sum_h sum_i A(h,i,j), A = row-wise softmax of the scaled logits
 * over the valid keys of the selected key blocks (Eq. 5), zero elsewhere.  marg: [B,N]. */
void usvo_key_marginal(const uint16_t* q, const int64_t* sq, const uint16_t* k, const int64_t* sk,
                       int B, int H, int N, int d, const int32_t* sel, const int32_t* k_per_head,
                       int kmax, double scale, double* marg) {
    int NB = (N + USVO_BS - 1) / USVO_BS;
    for (int64_t x = 0; x < (int64_t)B * N; ++x) marg[x] = 0.0;
    double* a = (double*)malloc(sizeof(double) * (size_t)N);
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int i = 0; i < N; ++i) {
                const int32_t* row = sel + (((int64_t)b * H + h) * NB + i / USVO_BS) * kmax;
                int nk = 0;
                double mx = -INFINITY;
                for (int t = 0; t < k_per_head[h]; ++t) {
                    int J = row[t];
                    if (J < 0) continue;
                    for (int j = J * USVO_BS; j < (J + 1) * USVO_BS && j < N; ++j) {
                        double acc = 0.0;
                        for (int e = 0; e < d; ++e)
                            acc += bf16_val(q[b * sq[0] + h * sq[1] + i * sq[2] + e]) *
                                   bf16_val(k[b * sk[0] + h * sk[1] + j * sk[2] + e]);
                        a[nk] = acc * scale;
                        idx[nk] = j;
                        mx = a[nk] > mx ? a[nk] : mx;
                        ++nk;
                    }
                }
                double sum = 0.0;
                for (int c = 0; c < nk; ++c) {
                    a[c] = exp(a[c] - mx);
                    sum += a[c];
                }
                for (int c = 0; c < nk; ++c) marg[(int64_t)b * N + idx[c]] += a[c] / sum;
            }
    for (int64_t x = 0; x < (int64_t)B * N; ++x) marg[x] /= (double)H * (double)N;
    free(a);
    free(idx);
}

/* Eq. 17: h = -(1/log N) sum_j abar(j) log abar(j), with 0 log 0 = 0. */
double usvo_entropy(const double* marg, int N) {
    double s = 0.0;
    for (int j = 0; j < N; ++j)
        if (marg[j] > 0.0) s -= marg[j] * log(marg[j]);
    return N > 1 ? s / log((double)N) : 0.0;
}

/* Eq. 18-19 for the L layers of one step. */
void usvo_allocate(const double* h, int L, double gamma, double rho_bar, double rho_min,
                   double rho_max, double* rho) {
    double mean = 0.0;
    for (int l = 0; l < L; ++l) mean += pow(1.0 - h[l], gamma);
    mean /= (double)L;
    for (int l = 0; l < L; ++l) {
        double w = pow(1.0 - h[l], gamma);
        double r = rho_bar * w / mean;
        rho[l] = r < rho_min ? rho_min : (r > rho_max ? rho_max : r);
    }
}
