/*
 * CPU oracle for paged-KV rollout attention.  TEST INFRASTRUCTURE ONLY: the
 * product (the CUDA library) never links, loads or calls anything in this file;
 * only the tests, the smoke check and the bench's CPU-baseline leg do.
 *
 * What it computes.  The paper treats the rollout engine step as a black box
 * (the inference worker's event loop runs one decode or prefill step at a time
 * over the requests it holds, Sec. 6.1) acting on trajectories whose context grows by one
 * (observation, action) pair per turn (Sec. 6.1, EnvManager) and whose decode
 * phase is bound by reading that whole context per generated token (Sec. 3.1).
 * The paper prints no formula for the step; the operation has a plain
 * definition, which is written out here and nothing more:
 *
 *   append : the r-th new row of trajectory t goes to logical position
 *            pos = len_before[t] + r, i.e. physical page table[t][pos / P],
 *            slot pos % P, for every kv head, as a bit copy.
 *   attend : query row with c visible keys, q head hq, kv head h = hq / g:
 *            s_j = scale * <q, k_j>, j in [j0, c);  m = max_j s_j;
 *            w_j = exp(s_j - m);  Z = sum_j w_j;
 *            out = sum_j w_j v_j / Z;   lse = m + ln Z.
 *   gather : the inverse of append, for handing a trajectory's cache to another worker
 *            (prefill/decode disaggregation, Sec. 6.3): row r of item i is the token at logical
 *            position r of trajectory t, copied bit for bit from its page slot.
 *   reserve: page bookkeeping between engine steps (Sec. 6.1: ADD / ABORT commands are processed
 *            between steps; Sec. 6.2: stale trajectories are evicted).  The free pages form a
 *            stack; item i, in item order, pops the pages that its trajectory needs to grow by
 *            new_tokens[i] and stores them in the next page-table entries.
 *   release: item i, in item order, pushes the pages its trajectory owns (logical order), marks
 *            the entries -1 and sets the length to 0.
 *   combine: parts (out_s, lse_s) over disjoint key ranges merge as
 *            M = max_s lse_s; a_s = exp(lse_s - M); out = sum a_s out_s / sum a_s;
 *            lse = M + ln sum a_s.
 *
 *   e4m3   : the 8-bit floating-point code of an fp8 KV pool (OCP 8-bit floating point specification, E4M3:
 *            1 sign, 4 exponent bits with bias 7, 3 mantissa bits; exponent field 0 holds the subnormals
 *            m/8 * 2^-6; there are no infinities and S.1111.111 is NaN, so the largest finite value is
 *            1.75 * 2^8 = 448).  encode rounds a float to the nearest code, ties to the even code, and
 *            saturates to +-448; decode returns the code's value.  A quantised append is encode applied
 *            to (row element * 1/scale), the product taken in fp32, followed by the plain bit-copy append.
 *
 * Everything floating point is fp64; bf16 inputs convert exactly.  No blocking,
 * no online softmax, no reordering: two passes over the keys, in index order.
 * Parity status: every function here is pinned by tests/test_oracle_pins.py, tests/test_oracle_pages.py or
 * tests/test_oracle_fp8.py
 * (closed forms, invariants, an independent dense routine, brute force).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_BAD_PAGE = 2, ORACLE_BAD_LENGTH = 3 };

static double bf16_to_f64(uint16_t bits) {
    uint32_t w = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Append.  seq_lens holds lengths BEFORE the call, indexed by trajectory; item i appends rows
 * new_indptr[i]..new_indptr[i+1] of k_new/v_new ([total_new][Hkv][D]) to trajectory
 * traj_ids[i] (identity when traj_ids is NULL).  seq_lens_out (nullable, indexed by
 * trajectory) receives len + n for the trajectories named; others are left untouched. */
int oracle_kv_append(uint16_t *k_pool, uint16_t *v_pool, int32_t num_pages, int32_t P, int32_t Hkv, int32_t D,
                     const int32_t *page_table, int32_t max_pages, const int32_t *seq_lens, int32_t num_traj,
                     const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items,
                     const uint16_t *k_new, const uint16_t *v_new, int32_t *seq_lens_out) {
    if (P <= 0 || Hkv <= 0 || D <= 0 || n_items < 0) return ORACLE_BAD_ARG;
    for (int32_t i = 0; i < n_items; ++i) {
        int32_t t = traj_ids ? traj_ids[i] : i;
        if (t < 0 || t >= num_traj) return ORACLE_BAD_ARG;
        int32_t n = new_indptr[i + 1] - new_indptr[i];
        int32_t len = seq_lens[t];
        if (n < 0 || len < 0) return ORACLE_BAD_LENGTH;
        for (int32_t r = 0; r < n; ++r) {
            int64_t pos = (int64_t)len + r;
            int64_t lp = pos / P;
            if (lp >= max_pages) return ORACLE_BAD_LENGTH;
            int32_t pg = page_table[(int64_t)t * max_pages + lp];
            if (pg < 0 || pg >= num_pages) return ORACLE_BAD_PAGE;
            int64_t slot = pos % P;
            int64_t row = (int64_t)new_indptr[i] + r;
            for (int32_t h = 0; h < Hkv; ++h) {
                int64_t dst = (((int64_t)pg * Hkv + h) * P + slot) * D;
                int64_t src = (row * Hkv + h) * D;
                memcpy(k_pool + dst, k_new + src, (size_t)D * sizeof(uint16_t));
                memcpy(v_pool + dst, v_new + src, (size_t)D * sizeof(uint16_t));
            }
        }
        if (seq_lens_out) seq_lens_out[t] = len + n;
    }
    return ORACLE_OK;
}

/* Gather.  Item i copies the first n_i = out_indptr[i+1] - out_indptr[i] tokens of trajectory
 * traj_ids[i] (identity when NULL) into rows out_indptr[i].. of k_out/v_out ([total][Hkv][D]).
 * n_i must not exceed the trajectory's length. */
int oracle_kv_gather(const uint16_t *k_pool, const uint16_t *v_pool, int32_t num_pages, int32_t P, int32_t Hkv, int32_t D,
                     const int32_t *page_table, int32_t max_pages, const int32_t *seq_lens, int32_t num_traj,
                     const int32_t *traj_ids, const int32_t *out_indptr, int32_t n_items, uint16_t *k_out, uint16_t *v_out) {
    if (P <= 0 || Hkv <= 0 || D <= 0 || n_items < 0) return ORACLE_BAD_ARG;
    for (int32_t i = 0; i < n_items; ++i) {
        int32_t t = traj_ids ? traj_ids[i] : i;
        if (t < 0 || t >= num_traj) return ORACLE_BAD_ARG;
        int32_t n = out_indptr[i + 1] - out_indptr[i];
        if (n < 0 || n > seq_lens[t]) return ORACLE_BAD_LENGTH;
        for (int32_t r = 0; r < n; ++r) {
            int64_t lp = r / P;
            if (lp >= max_pages) return ORACLE_BAD_LENGTH;
            int32_t pg = page_table[(int64_t)t * max_pages + lp];
            if (pg < 0 || pg >= num_pages) return ORACLE_BAD_PAGE;
            int64_t row = (int64_t)out_indptr[i] + r;
            for (int32_t h = 0; h < Hkv; ++h) {
                int64_t src = (((int64_t)pg * Hkv + h) * P + r % P) * D;
                int64_t dst = (row * Hkv + h) * D;
                memcpy(k_out + dst, k_pool + src, (size_t)D * sizeof(uint16_t));
                memcpy(v_out + dst, v_pool + src, (size_t)D * sizeof(uint16_t));
            }
        }
    }
    return ORACLE_OK;
}

/* Reserve.  free_pages[0 .. *free_count) is the stack (top at the end).  Returns ORACLE_BAD_LENGTH and
 * changes nothing when the stack is too small or a trajectory would outgrow its page-table row. */
int oracle_pages_reserve(int32_t *free_pages, int32_t *free_count, int32_t P, int32_t *page_table, int32_t max_pages,
                         const int32_t *seq_lens, int32_t num_traj, const int32_t *traj_ids, const int32_t *new_tokens,
                         int32_t n_items) {
    if (P <= 0 || n_items < 0) return ORACLE_BAD_ARG;
    int64_t need_total = 0;
    for (int32_t i = 0; i < n_items; ++i) {
        int32_t t = traj_ids ? traj_ids[i] : i;
        if (t < 0 || t >= num_traj || new_tokens[i] < 0 || seq_lens[t] < 0) return ORACLE_BAD_ARG;
        int64_t have = ((int64_t)seq_lens[t] + P - 1) / P;
        int64_t want = ((int64_t)seq_lens[t] + new_tokens[i] + P - 1) / P;
        if (want > max_pages) return ORACLE_BAD_LENGTH;
        need_total += want - have;
    }
    if (need_total > *free_count) return ORACLE_BAD_LENGTH;
    int32_t top = *free_count;
    for (int32_t i = 0; i < n_items; ++i) {
        int32_t t = traj_ids ? traj_ids[i] : i;
        int64_t have = ((int64_t)seq_lens[t] + P - 1) / P;
        int64_t want = ((int64_t)seq_lens[t] + new_tokens[i] + P - 1) / P;
        for (int64_t lp = have; lp < want; ++lp) page_table[(int64_t)t * max_pages + lp] = free_pages[--top];
    }
    *free_count = top;
    return ORACLE_OK;
}

/* Release.  seq_lens is updated in place (0 for the trajectories named). */
int oracle_pages_release(int32_t *free_pages, int32_t *free_count, int32_t capacity, int32_t P, int32_t *page_table,
                         int32_t max_pages, int32_t *seq_lens, int32_t num_traj, const int32_t *traj_ids, int32_t n_items) {
    if (P <= 0 || n_items < 0) return ORACLE_BAD_ARG;
    int64_t total = *free_count;
    for (int32_t i = 0; i < n_items; ++i) {
        int32_t t = traj_ids ? traj_ids[i] : i;
        if (t < 0 || t >= num_traj || seq_lens[t] < 0) return ORACLE_BAD_ARG;
        int64_t have = ((int64_t)seq_lens[t] + P - 1) / P;
        if (have > max_pages) return ORACLE_BAD_LENGTH;
        total += have;
    }
    if (total > capacity) return ORACLE_BAD_LENGTH;
    int32_t top = *free_count;
    for (int32_t i = 0; i < n_items; ++i) {
        int32_t t = traj_ids ? traj_ids[i] : i;
        int64_t have = ((int64_t)seq_lens[t] + P - 1) / P;
        for (int64_t lp = 0; lp < have; ++lp) {
            free_pages[top++] = page_table[(int64_t)t * max_pages + lp];
            page_table[(int64_t)t * max_pages + lp] = -1;
        }
        seq_lens[t] = 0;
    }
    *free_count = top;
    return ORACLE_OK;
}

/* Stale eviction (Sec. 6.2, asynchronous bound alpha).  With the agent LLM at version n, a buffered trajectory must
 * have been initiated by a version no older than n - alpha; the ones outside this window are aborted.  Here: every
 * live trajectory (len > 0) with start_version[t] < n - alpha gives its pages back, exactly as oracle_pages_release
 * does for the list of those trajectories in ascending order; evicted_ids receives that list, *n_evicted its length. */
int oracle_pages_evict_stale(int32_t *free_pages, int32_t *free_count, int32_t capacity, int32_t P, int32_t *page_table,
                             int32_t max_pages, int32_t *seq_lens, int32_t num_traj, const int32_t *start_version,
                             int32_t current_version, int32_t alpha, int32_t *evicted_ids, int32_t *n_evicted) {
    if (P <= 0 || num_traj < 0) return ORACLE_BAD_ARG;
    int32_t n = 0;
    for (int32_t t = 0; t < num_traj; ++t) {
        if (seq_lens[t] < 0) return ORACLE_BAD_ARG;
        if (seq_lens[t] > 0 && (int64_t)start_version[t] < (int64_t)current_version - (int64_t)alpha) evicted_ids[n++] = t;
    }
    int rc = oracle_pages_release(free_pages, free_count, capacity, P, page_table, max_pages, seq_lens, num_traj, evicted_ids, n);
    if (rc != ORACLE_OK) return rc;
    *n_evicted = n;
    return ORACLE_OK;
}

/* Attention of n_rows query rows.  Row r belongs to trajectory row_traj[r] and sees keys
 * row_begin[r] <= j < row_count[r] of that trajectory (row_begin NULL = 0).  q is
 * [n_rows][Hq][D] bf16; out is [n_rows][Hq][D] fp64, lse [n_rows][Hq] fp64 (natural log).
 * An empty key range gives out = 0, lse = -inf. */
int oracle_attend(const uint16_t *k_pool, const uint16_t *v_pool, int32_t num_pages, int32_t P, int32_t Hkv, int32_t D,
                  const int32_t *page_table, int32_t max_pages, int32_t num_traj,
                  int64_t n_rows, const int32_t *row_traj, const int32_t *row_begin, const int32_t *row_count,
                  const uint16_t *q, int32_t Hq, float sm_scale, double *out, double *lse) {
    if (P <= 0 || Hkv <= 0 || D <= 0 || Hq <= 0 || Hq % Hkv != 0 || n_rows < 0) return ORACLE_BAD_ARG;
    const int32_t g = Hq / Hkv;
    const double scale = (double)sm_scale;
    int status = ORACLE_OK;
    /* validate first, so the parallel region has nothing to report */
    for (int64_t r = 0; r < n_rows; ++r) {
        int32_t t = row_traj[r];
        if (t < 0 || t >= num_traj) return ORACLE_BAD_ARG;
        int32_t c = row_count[r], j0 = row_begin ? row_begin[r] : 0;
        if (c < 0 || j0 < 0) return ORACLE_BAD_LENGTH;
        if (c > 0 && (int64_t)(c - 1) / P >= max_pages) return ORACLE_BAD_LENGTH;
        for (int64_t lp = j0 / P; c > j0 && lp * P < c; ++lp) {
            int32_t pg = page_table[(int64_t)t * max_pages + lp];
            if (pg < 0 || pg >= num_pages) return ORACLE_BAD_PAGE;
        }
    }
    const int64_t n_work = n_rows * Hq;
#pragma omp parallel
    {
        double *s = NULL;
        size_t s_cap = 0;
        double *qd = (double *)malloc((size_t)D * sizeof(double));
        double *acc = (double *)malloc((size_t)D * sizeof(double));
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < n_work; ++w) {
            int64_t r = w / Hq;
            int32_t hq = (int32_t)(w % Hq);
            int32_t h = hq / g;
            int32_t t = row_traj[r];
            int32_t c = row_count[r], j0 = row_begin ? row_begin[r] : 0;
            double *o = out + (r * Hq + hq) * D;
            for (int32_t d = 0; d < D; ++d) o[d] = 0.0;
            if (c <= j0) { lse[r * Hq + hq] = -INFINITY; continue; }
            size_t n = (size_t)(c - j0);
            if (n > s_cap) { free(s); s = (double *)malloc(n * sizeof(double)); s_cap = n; }
            const uint16_t *qp = q + (r * Hq + hq) * D;
            for (int32_t d = 0; d < D; ++d) qd[d] = bf16_to_f64(qp[d]);
            double m = -INFINITY;
            for (int32_t j = j0; j < c; ++j) {
                int32_t pg = page_table[(int64_t)t * max_pages + j / P];
                const uint16_t *kp = k_pool + (((int64_t)pg * Hkv + h) * P + j % P) * D;
                double dot = 0.0;
                for (int32_t d = 0; d < D; ++d) dot += qd[d] * bf16_to_f64(kp[d]);
                double sj = scale * dot;
                s[j - j0] = sj;
                if (sj > m) m = sj;
            }
            double Z = 0.0;
            for (int32_t d = 0; d < D; ++d) acc[d] = 0.0;
            for (int32_t j = j0; j < c; ++j) {
                int32_t pg = page_table[(int64_t)t * max_pages + j / P];
                const uint16_t *vp = v_pool + (((int64_t)pg * Hkv + h) * P + j % P) * D;
                double wj = exp(s[j - j0] - m);
                Z += wj;
                for (int32_t d = 0; d < D; ++d) acc[d] += wj * bf16_to_f64(vp[d]);
            }
            for (int32_t d = 0; d < D; ++d) o[d] = acc[d] / Z;
            lse[r * Hq + hq] = m + log(Z);
        }
        free(s); free(qd); free(acc);
    }
    return status;
}

/* Merge n_parts partial results of ONE (row, head): parts_out [n_parts][D], parts_lse [n_parts].
 * Parts with lse = -inf (empty ranges) contribute nothing; all empty gives out = 0, lse = -inf. */
int oracle_lse_combine(int32_t n_parts, int32_t D, const double *parts_out, const double *parts_lse,
                       double *out, double *lse) {
    if (n_parts < 0 || D <= 0) return ORACLE_BAD_ARG;
    double M = -INFINITY;
    for (int32_t s = 0; s < n_parts; ++s) if (parts_lse[s] > M) M = parts_lse[s];
    for (int32_t d = 0; d < D; ++d) out[d] = 0.0;
    if (M == -INFINITY) { *lse = -INFINITY; return ORACLE_OK; }
    double A = 0.0;
    for (int32_t s = 0; s < n_parts; ++s) {
        double a = exp(parts_lse[s] - M);
        A += a;
        for (int32_t d = 0; d < D; ++d) out[d] += a * parts_out[(int64_t)s * D + d];
    }
    for (int32_t d = 0; d < D; ++d) out[d] /= A;
    *lse = M + log(A);
    return ORACLE_OK;
}

/* E4M3 decode: value of each code as a double (NaN for 0x7f / 0xff). */
int oracle_e4m3_decode(const uint8_t *codes, int64_t n, double *out) {
    for (int64_t i = 0; i < n; ++i) {
        const int c = codes[i];
        const int e = (c >> 3) & 15, m = c & 7;
        double v;
        if (e == 15 && m == 7) v = NAN;
        else if (e == 0) v = ldexp((double)m / 8.0, -6);
        else v = ldexp(1.0 + (double)m / 8.0, e - 7);
        out[i] = (c & 0x80) ? -v : v;
    }
    return ORACLE_OK;
}

/* E4M3 encode: nearest code, ties to even, magnitudes of 448 and above (and infinities) give +-448, NaN gives 0x7f. */
int oracle_e4m3_encode(const float *x, int64_t n, uint8_t *codes) {
    for (int64_t i = 0; i < n; ++i) {
        const float f = x[i];
        if (isnan(f)) { codes[i] = 0x7f; continue; }
        const uint8_t sign = signbit(f) ? 0x80 : 0x00;
        const double a = fabs((double)f);
        uint8_t mag;
        if (a >= 448.0) {
            mag = 0x7e;
        } else if (a < ldexp(1.0, -6)) {
            /* subnormal range: multiples of 2^-9; 8 of them is the smallest normal, code 0x08 */
            mag = (uint8_t)nearbyint(ldexp(a, 9));
        } else {
            int e;
            const double fr = frexp(a, &e);          /* a = fr * 2^e, fr in [0.5, 1) */
            int ex = e - 1;                           /* a = (2 fr) * 2^ex, 2 fr in [1, 2) */
            int m = (int)nearbyint((2.0 * fr - 1.0) * 8.0);
            if (m == 8) { m = 0; ex += 1; }
            const int code = ((ex + 7) << 3) | m;
            mag = code > 0x7e ? 0x7e : (uint8_t)code;
        }
        codes[i] = sign | mag;
    }
    return ORACLE_OK;
}
