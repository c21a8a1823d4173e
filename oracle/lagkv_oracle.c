/*
 * LagKV compress pass -- float64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * LagKV compression pass (arXiv 2504.04704, Section 2.2 "LagKV") computes.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline leg to
 * check the CUDA library; the CUDA library never calls it and shares no code with it.
 *
 * Every step is written in the order the paper's Methodology lists it, one loop per
 * step, with no blocking, fusion or reordering.  Inputs are 16-bit patterns
 * (uint16_t) in the cache's storage format, bf16 (the default), IEEE fp16, or an fp8 e4m3 byte
 * zero-extended to 16 bits; each is
 * widened exactly to double before any arithmetic.  The paper does not name a storage
 * format; the method is the same for either.
 *
 * Readings taken where the paper leaves a choice:
 *   - min/max are taken over the tokens of the reference partition, one pair per
 *     channel (Eq. 7, Eq. 8 reduce over the sequence axis).
 *   - "Std." is the standard deviation over the head_dim channels of one token,
 *     two-pass, divisor (D - ddof); ddof is a parameter (1 = sample std, 0 =
 *     population std).  The paper does not say which: PARITY UNPINNED for ddof.
 *   - Softmax (Eq. 10) runs over the L tokens of the partition, separately for K and V.
 *   - A channel whose reference range max-min is zero contributes y = 0 for every
 *     token (no epsilon).  The paper does not cover this: PARITY UNPINNED.
 *   - Values outside the reference range are not clamped.
 *   - keep count k = ceil(r*L), clamped to [1, L]; non-integer r*L is not covered
 *     by the paper: PARITY UNPINNED off the integer case.
 *   - Score ties keep the lower index; kept rows stay in ascending position order.
 *   - Scoring variants of Section 4.3: LocalKV takes min/max from the partition
 *     itself (Eq. 14, Eq. 15); the L2 variant scores a token by minus the Euclidean
 *     norm of its key (Eq. 16).
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC -o liblagkv_oracle.so lagkv_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { LAGKV_ORACLE_LAGKV = 0, LAGKV_ORACLE_LOCALKV = 1, LAGKV_ORACLE_L2NORM = 2 };

enum { LAGKV_ORACLE_BF16 = 0, LAGKV_ORACLE_FP16 = 1, LAGKV_ORACLE_FP8_E4M3 = 2 };

/* bf16 bit pattern -> double, exact (bf16 is the upper half of an IEEE binary32). */
static double bf16_to_double(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* IEEE binary16 bit pattern -> double, exact: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double fp16_to_double(uint16_t bits)
{
    int sign = bits >> 15, e = (bits >> 10) & 31, frac = bits & 1023;
    double v;
    if (e == 0)
        v = ldexp((double)frac, -24);                 /* zero and subnormals */
    else if (e == 31)
        v = frac ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)frac / 1024.0, e - 15);
    return sign ? -v : v;
}

/* fp8 "e4m3fn" byte -> double, exact: 1 sign, 4 exponent (bias 7), 3 fraction bits; the format
 * has no infinities, and exponent 15 with fraction 7 (0x7f, 0xff) is its only NaN.  The byte sits
 * in the low half of the 16-bit element the oracle's arrays carry (the caller zero-extends). */
static double fp8_e4m3_to_double(uint16_t bits)
{
    int sign = (bits >> 7) & 1, e = (bits >> 3) & 15, frac = bits & 7;
    double v;
    if (e == 0)
        v = ldexp((double)frac, -9);                  /* zero and subnormals: frac/8 * 2^-6 */
    else if (e == 15 && frac == 7)
        v = NAN;
    else
        v = ldexp(1.0 + (double)frac / 8.0, e - 7);
    return sign ? -v : v;
}

/* The storage format of the cache is the only place a value's bits are interpreted. */
static double decode(uint16_t bits, int storage)
{
    if (storage == LAGKV_ORACLE_FP8_E4M3) return fp8_e4m3_to_double(bits);
    return storage == LAGKV_ORACLE_FP16 ? fp16_to_double(bits) : bf16_to_double(bits);
}

/* out[i] = value of bits[i] in the given storage format (exposed so that tests can pin it). */
void lagkv_oracle_decode(const uint16_t *bits, int64_t n, int storage, double *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = decode(bits[i], storage);
}

int lagkv_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void lagkv_oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Retained tokens per partition: r*L of the L tokens stay (text before Eq. 12). */
int64_t lagkv_oracle_keep_count(double r, int64_t L)
{
    int64_t k = (int64_t)ceil(r * (double)L - 1e-9);
    if (k < 1) k = 1;
    if (k > L) k = L;
    return k;
}

/*
 * Length after one pass over a cache of seq_len rows whose first static_len rows
 * (sink + already compressed part) are left alone.  With static_len = S this is
 * Eq. 12:  L_R = S + rL*(floor((Ls-S)/L) - 1) + L + Mod(Ls-S, L);
 * below 2L of remaining rows the pass is skipped (third bullet of Section 2.2,
 * and the remark after Eq. 13 that shorter sequences are not compressed at all).
 */
int64_t lagkv_oracle_compressed_len(int64_t seq_len, int64_t static_len, int64_t L, int64_t k)
{
    int64_t rest = seq_len - static_len;
    if (rest < 2 * L) return seq_len;
    int64_t n = rest / L;
    int64_t rem = rest % L;
    return static_len + k * (n - 1) + L + rem;
}

/*
 * score(Z) of Eq. 10 for one tensor of one partition.
 *   cur, ref : [L, D] rows of 16-bit values, row_stride elements apart
 *   out      : [L] softmax(Std(normalised cur))
 */
static void tensor_score(const uint16_t *cur, const uint16_t *ref, int64_t L, int64_t D,
                         int64_t row_stride, int ddof, int storage, double *out)
{
    double *mn = (double *)malloc(sizeof(double) * (size_t)D);
    double *mx = (double *)malloc(sizeof(double) * (size_t)D);
    double *y = (double *)malloc(sizeof(double) * (size_t)D);
    double *sd = (double *)malloc(sizeof(double) * (size_t)L);

    /* Eq. 7 and Eq. 8: per channel, min and max over the reference tokens. */
    for (int64_t c = 0; c < D; ++c) {
        mn[c] = decode(ref[c], storage);
        mx[c] = mn[c];
        for (int64_t t = 1; t < L; ++t) {
            double z = decode(ref[t * row_stride + c], storage);
            if (z < mn[c]) mn[c] = z;
            if (z > mx[c]) mx[c] = z;
        }
    }

    for (int64_t t = 0; t < L; ++t) {
        /* Eq. 9: min-max normalisation of the current token, channel by channel. */
        for (int64_t c = 0; c < D; ++c) {
            double z = decode(cur[t * row_stride + c], storage);
            double range = mx[c] - mn[c];
            y[c] = (range > 0.0) ? (z - mn[c]) / range : 0.0;
        }
        /* Std. of Eq. 10: over the D channels of this token, two passes. */
        double mean = 0.0;
        for (int64_t c = 0; c < D; ++c) mean += y[c];
        mean /= (double)D;
        double ss = 0.0;
        for (int64_t c = 0; c < D; ++c) ss += (y[c] - mean) * (y[c] - mean);
        sd[t] = sqrt(ss / (double)(D - ddof));
    }

    /* Softmax of Eq. 10: over the L tokens of the partition. */
    double top = sd[0];
    for (int64_t t = 1; t < L; ++t)
        if (sd[t] > top) top = sd[t];
    double denom = 0.0;
    for (int64_t t = 0; t < L; ++t) {
        out[t] = exp(sd[t] - top);
        denom += out[t];
    }
    for (int64_t t = 0; t < L; ++t) out[t] /= denom;

    free(mn);
    free(mx);
    free(y);
    free(sd);
}

/*
 * Final per-token score of one partition.
 *   variant 0 (LagKV)  : Eq. 11, score(K) + score(V), reference = next partition.
 *   variant 1 (LocalKV): same, reference = the partition itself (Eq. 14, Eq. 15);
 *                        the caller passes ref == cur.
 *   variant 2 (L2 norm): Eq. 16, minus the Euclidean norm of the key row.
 * sK, sV may be NULL; when given they receive the two summands (variants 0, 1).
 */
void lagkv_oracle_partition_scores(const uint16_t *Kcur, const uint16_t *Vcur,
                                   const uint16_t *Kref, const uint16_t *Vref, int64_t L,
                                   int64_t D, int64_t row_stride, int ddof, int variant,
                                   int storage, double *score, double *sK, double *sV)
{
    if (variant == LAGKV_ORACLE_L2NORM) {
        for (int64_t t = 0; t < L; ++t) {
            double ss = 0.0;
            for (int64_t c = 0; c < D; ++c) {
                double z = decode(Kcur[t * row_stride + c], storage);
                ss += z * z;
            }
            score[t] = -sqrt(ss);
        }
        return;
    }
    double *a = (double *)malloc(sizeof(double) * (size_t)L);
    double *b = (double *)malloc(sizeof(double) * (size_t)L);
    tensor_score(Kcur, Kref, L, D, row_stride, ddof, storage, a);
    tensor_score(Vcur, Vref, L, D, row_stride, ddof, storage, b);
    for (int64_t t = 0; t < L; ++t) score[t] = a[t] + b[t]; /* Eq. 11 */
    if (sK) memcpy(sK, a, sizeof(double) * (size_t)L);
    if (sV) memcpy(sV, b, sizeof(double) * (size_t)L);
    free(a);
    free(b);
}

/*
 * Top-k of one partition (last bullet of Section 2.2): the k largest scores, a tie
 * going to the lower index; the result is listed in ascending index order.
 * Plain selection, O(k*L).
 */
void lagkv_oracle_topk(const double *score, int64_t L, int64_t k, int32_t *idx_out)
{
    char *taken = (char *)calloc((size_t)L, 1);
    for (int64_t j = 0; j < k; ++j) {
        int64_t best = -1;
        for (int64_t t = 0; t < L; ++t) {
            if (taken[t]) continue;
            if (best < 0 || score[t] > score[best]) best = t; /* strict: lower index wins */
        }
        if (best < 0) break; /* k > L: every token is already taken */
        taken[best] = 1;
    }
    int64_t w = 0;
    for (int64_t t = 0; t < L; ++t)
        if (taken[t]) idx_out[w++] = (int32_t)t;
    free(taken);
}

/*
 * One compress pass over contiguous caches K, V of shape [B, H, seq_len, D] (16-bit patterns).
 * The first static_len rows of every (b, h) are the sink plus the already compressed
 * part and are copied through; the rest is cut into partitions of L rows, partition p
 * is scored against partition p+1, k rows of it are kept, and the last full partition
 * together with the Mod(rest, L) trailing rows forms the sliding window.
 *
 * Outputs (any may be NULL):
 *   idx_out    [B, H, L_R]        source row of every output row
 *   K_out,V_out[B, H, L_R, D]     the compacted cache
 *   scores_out [B, H, (n-1)*L]    final score of every token of a compressed partition
 * Returns L_R.
 */
int64_t lagkv_oracle_compress(const uint16_t *K, const uint16_t *V, int64_t B, int64_t H,
                              int64_t seq_len, int64_t D, int64_t static_len, int64_t L,
                              int64_t k, int ddof, int variant, int storage, int32_t *idx_out,
                              uint16_t *K_out, uint16_t *V_out, double *scores_out)
{
    int64_t L_R = lagkv_oracle_compressed_len(seq_len, static_len, L, k);
    int64_t rest = seq_len - static_len;
    int64_t n = (rest >= 2 * L) ? rest / L : 0; /* partitions; 0 = pass skipped */
    int64_t n_c = (n > 0) ? n - 1 : 0;          /* compressed partitions      */

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t u = 0; u < B * H; ++u) {
        const uint16_t *Ku = K + u * seq_len * D;
        const uint16_t *Vu = V + u * seq_len * D;
        int32_t *src = (int32_t *)malloc(sizeof(int32_t) * (size_t)L_R);
        int64_t w = 0;

        /* static part: attention sink and already compressed rows stay */
        for (int64_t t = 0; t < static_len && n > 0; ++t) src[w++] = (int32_t)t;

        if (n == 0) {
            for (int64_t t = 0; t < seq_len; ++t) src[w++] = (int32_t)t;
        } else {
            double *score = (double *)malloc(sizeof(double) * (size_t)L);
            int32_t *keep = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
            for (int64_t p = 0; p < n_c; ++p) {
                int64_t cur = static_len + p * L;
                int64_t ref = (variant == LAGKV_ORACLE_LOCALKV) ? cur : cur + L;
                lagkv_oracle_partition_scores(Ku + cur * D, Vu + cur * D, Ku + ref * D,
                                              Vu + ref * D, L, D, D, ddof, variant, storage,
                                              score, NULL, NULL);
                if (scores_out)
                    memcpy(scores_out + (u * n_c + p) * L, score, sizeof(double) * (size_t)L);
                lagkv_oracle_topk(score, L, k, keep);
                for (int64_t j = 0; j < k; ++j) src[w++] = (int32_t)(cur + keep[j]);
            }
            /* sliding window: last full partition plus the remainder */
            for (int64_t t = static_len + n_c * L; t < seq_len; ++t) src[w++] = (int32_t)t;
            free(score);
            free(keep);
        }

        for (int64_t j = 0; j < L_R; ++j) {
            if (idx_out) idx_out[u * L_R + j] = src[j];
            if (K_out) memcpy(K_out + (u * L_R + j) * D, Ku + (int64_t)src[j] * D, 2 * (size_t)D);
            if (V_out) memcpy(V_out + (u * L_R + j) * D, Vu + (int64_t)src[j] * D, 2 * (size_t)D);
        }
        free(src);
    }
    return L_R;
}

/* Row gather: out[u, j, :] = in[u, idx[u, j], :] for every (b, h) unit u. */
void lagkv_oracle_gather(const uint16_t *in, int64_t units, int64_t seq_len, int64_t D,
                         const int32_t *idx, int64_t n_idx, uint16_t *out)
{
    for (int64_t u = 0; u < units; ++u)
        for (int64_t j = 0; j < n_idx; ++j)
            memcpy(out + (u * n_idx + j) * D, in + (u * seq_len + idx[u * n_idx + j]) * D,
                   2 * (size_t)D);
}
