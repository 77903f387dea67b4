/*
 * Tiled Bit Networks -- CPU oracle (TEST INFRASTRUCTURE, not the product).
 *
 * A plain, slow, obviously-correct restatement of what one tiled layer computes,
 * written from the paper's Section 3 (Eq. 1-8) and Section 5.1 (Algorithm 1).
 * It exists so that the CUDA library can be checked against something that
 * shares no code with it.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the library itself never does.
 *
 * Conventions (every one is a reading of the paper, listed in the design notes):
 *   N      number of elements of the layer's weight tensor            (Sec. 3)
 *   p      compression factor = number of times the tile is repeated  (Sec. 3)
 *   q=N/p  tile length                                                (Sec. 3)
 *   flat index f is the row-major (C order) index of the weight tensor:
 *          (out,in) for fully-connected, (Cout,Cin,kh,kw) for convolution.
 *   W* (Eq. 1) is the row-major p x q view of the flat tensor: W*[j][i] = W[j*q+i].
 *
 * Arithmetic: the chunk-sum of Eq. 2 is a sequential fp32 sum in increasing j
 * (its sign decides a bit, so the order and precision are part of the contract);
 * everything else accumulates in fp64.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py against
 * closed forms, library routines, brute force and the numbers the paper prints.
 *
 * Build: gcc -O2 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_ACT_NONE = 0, ORACLE_ACT_RELU = 1, ORACLE_ACT_GELU = 2 };

int tbn_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static double apply_act(double v, int act)
{
    if (act == ORACLE_ACT_RELU) return v > 0.0 ? v : 0.0;           /* Algorithm 1: fused ReLU */
    if (act == ORACLE_ACT_GELU) return 0.5 * v * (1.0 + erf(v * 0.70710678118654752440)); /* exact erf form */
    return v;
}

/*
 * Eq. 1-3: reshape W to p x q, sum over the p dimension, threshold.
 *   s_i = sum_{j<p} W[j*q + i]   (fp32, sequential in j)
 *   t_i = +1 if s_i > 0 else -1  (zero, negative zero and NaN all give -1)
 * bits[i] receives 1 for t_i = +1 and 0 for t_i = -1.
 * *sign_mismatch (nullable) counts the i whose fp64 sum has a different sign
 * decision: a diagnostic for near-cancelling sums, not part of the result.
 * Returns 0, or -1 when p does not divide N (Sec. 3 requires p*q = N).
 */
int tbn_oracle_aggregate(const float *W, int64_t N, int32_t p, uint8_t *bits, int64_t *sign_mismatch)
{
    if (p <= 0 || N < 0 || N % p != 0) return -1;
    const int64_t q = N / p;
    int64_t mism = 0;
    for (int64_t i = 0; i < q; ++i) {
        volatile float s = 0.0f;   /* volatile: force one fp32 rounding per add */
        double s64 = 0.0;
        for (int32_t j = 0; j < p; ++j) {
            s = s + W[(int64_t)j * q + i];
            s64 += (double)W[(int64_t)j * q + i];
        }
        const uint8_t b = (s > 0.0f) ? 1 : 0;
        bits[i] = b;
        if (b != ((s64 > 0.0) ? 1 : 0)) ++mism;
    }
    if (sign_mismatch) *sign_mismatch = mism;
    return 0;
}

/*
 * Eq. 6 (per layer) and Eq. 7-8 (per tile).  S is W, or the separate tensor A.
 *   per layer: alpha    = ||S||_1 / N
 *   per tile : alpha_j  = ||S[j*q .. (j+1)*q)||_1 / q,  j < p
 * fp64 accumulation, one rounding to fp32 at the end.
 */
int tbn_oracle_alpha(const float *S, int64_t N, int32_t p, int per_tile, float *alpha)
{
    if (p <= 0 || N < 0 || N % p != 0) return -1;
    const int64_t q = N / p;
    if (!per_tile) {
        double a = 0.0;
        for (int64_t f = 0; f < N; ++f) a += fabs((double)S[f]);
        alpha[0] = (float)(a / (double)N);
        return 0;
    }
    for (int32_t j = 0; j < p; ++j) {
        double a = 0.0;
        for (int64_t c = 0; c < q; ++c) a += fabs((double)S[(int64_t)j * q + c]);
        alpha[j] = (float)(a / (double)q);
    }
    return 0;
}

/*
 * Sec. 5.1: the tile is stored one bit per element.  Bit i of the tile is bit
 * (i mod 32) of 32-bit word (i div 32), least significant first; unused bits of
 * the last words are 0.  nwords is the size of the destination in words.
 * src > 0 gives bit 1, everything else bit 0 (the rule of Eq. 3).
 */
void tbn_oracle_pack(const float *src, int64_t q, uint32_t *words, int64_t nwords)
{
    for (int64_t w = 0; w < nwords; ++w) words[w] = 0u;
    for (int64_t i = 0; i < q; ++i)
        if (src[i] > 0.0f) words[i >> 5] |= (uint32_t)1u << (i & 31);
}

void tbn_oracle_pack_bits(const uint8_t *bits, int64_t q, uint32_t *words, int64_t nwords)
{
    for (int64_t w = 0; w < nwords; ++w) words[w] = 0u;
    for (int64_t i = 0; i < q; ++i)
        if (bits[i]) words[i >> 5] |= (uint32_t)1u << (i & 31);
}

/*
 * Eq. 4-5 and the scaling paragraph after Eq. 8: b = 1_p (x) t, B = vec^-1(b),
 * B_hat = alpha (.) B.   B_hat[f] = alpha_{f div q} * (bit[f mod q] ? +1 : -1),
 * with a single alpha when per_tile == 0.
 */
int tbn_oracle_expand(const uint32_t *words, int64_t N, int32_t p, const float *alpha, int per_tile,
                      float *B_hat)
{
    if (p <= 0 || N < 0 || N % p != 0) return -1;
    const int64_t q = N / p;
    for (int64_t f = 0; f < N; ++f) {
        const int64_t i = f % q;
        const int64_t j = f / q;
        const float t = ((words[i >> 5] >> (i & 31)) & 1u) ? 1.0f : -1.0f;
        const float a = per_tile ? alpha[j] : alpha[0];
        B_hat[f] = a * t;
    }
    return 0;
}

/*
 * Full-precision tiled weights (Sec. 5.2, the "FP, Tiled" kernel of Table 7): the same
 * replication and reshaping as Eq. 4-5, but the tile holds real values and is used as it is,
 * no threshold and no scaling factor:  B[f] = t[f mod q],  q = N / p.
 */
int tbn_oracle_expand_fp(const float *tile, int64_t N, int32_t p, float *B)
{
    if (p <= 0 || N < 0 || N % p != 0) return -1;
    const int64_t q = N / p;
    for (int64_t f = 0; f < N; ++f) B[f] = tile[f % q];
    return 0;
}

/*
 * Fully-connected layer with an explicit (already expanded) weight:
 *   y[b][i] = act( sum_{j<n} B_hat[i][j] * x[b][j] + bias[i] ),  j increasing, fp64.
 * x: T x n row-major, B_hat: m x n row-major (out x in), y: T x m row-major.
 */
void tbn_oracle_linear(const double *x, int64_t T, int32_t n, int32_t m, const float *B_hat,
                       const double *bias, int act, double *y)
{
    const int64_t total = T * (int64_t)m;
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < total; ++o) {
        const int64_t b = o / m;
        const int32_t i = (int32_t)(o % m);
        double acc = 0.0;
        for (int32_t j = 0; j < n; ++j)
            acc += (double)B_hat[(int64_t)i * n + j] * x[b * n + j];
        if (bias) acc += bias[i];
        y[o] = apply_act(acc, act);
    }
}

/*
 * Algorithm 1 (Sec. 5.1), the index-walk form, written independently of the
 * expand-then-multiply routine above: one pass over the flat weight index, a
 * tile index that returns to 0 when it has consumed q entries, and an alpha
 * index that advances at each such wrap.  tile holds +1/-1 values, q of them;
 * alpha holds p values (pass the same value p times for a single alpha).
 * The wrap is taken when the NEXT index would be q (the listing's test is off
 * by one); the walk runs across row ends, as the listing's does.
 */
void tbn_oracle_linear_alg1(const double *x, int64_t T, int32_t n, int32_t m, const float *tile,
                            int64_t q, const float *alpha, int relu, double *y)
{
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < T; ++b) {
        int64_t t_i = 0;
        int64_t a_i = 0;
        for (int32_t i = 0; i < m; ++i) {
            double acc = 0.0;
            for (int32_t j = 0; j < n; ++j) {
                acc += (double)tile[t_i] * x[b * n + j] * (double)alpha[a_i];
                if (t_i + 1 == q) { t_i = 0; ++a_i; } else { ++t_i; }
            }
            y[b * m + i] = relu ? (acc > 0.0 ? acc : 0.0) : acc;
        }
    }
}

/*
 * Convolution with an explicit weight: direct cross-correlation (no kernel flip),
 * zero padding, square stride, no dilation, one group.
 *   y[b][co][oh][ow] = act( sum_{ci,u,v} B_hat[co][ci][u][v] *
 *                           x[b][ci][oh*s+u-pad][ow*s+v-pad] + bias[co] )
 * x: NCHW, B_hat: (Cout,Cin,kh,kw) row-major, y: (Nb,Cout,Ho,Wo).
 */
void tbn_oracle_conv2d(const double *x, int32_t Nb, int32_t Cin, int32_t H, int32_t Wd,
                       int32_t Cout, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                       const float *B_hat, const double *bias, int act, double *y)
{
    const int32_t Ho = (H + 2 * pad - kh) / stride + 1;
    const int32_t Wo = (Wd + 2 * pad - kw) / stride + 1;
    const int64_t total = (int64_t)Nb * Cout;
#pragma omp parallel for schedule(static)
    for (int64_t bc = 0; bc < total; ++bc) {
        const int32_t b = (int32_t)(bc / Cout);
        const int32_t co = (int32_t)(bc % Cout);
        for (int32_t oh = 0; oh < Ho; ++oh) {
            for (int32_t ow = 0; ow < Wo; ++ow) {
                double acc = 0.0;
                for (int32_t ci = 0; ci < Cin; ++ci) {
                    for (int32_t u = 0; u < kh; ++u) {
                        for (int32_t v = 0; v < kw; ++v) {
                            const int32_t ih = oh * stride + u - pad;
                            const int32_t iw = ow * stride + v - pad;
                            if (ih < 0 || ih >= H || iw < 0 || iw >= Wd) continue;
                            const double w =
                                (double)B_hat[(((int64_t)co * Cin + ci) * kh + u) * kw + v];
                            acc += w * x[(((int64_t)b * Cin + ci) * H + ih) * Wd + iw];
                        }
                    }
                }
                if (bias) acc += bias[co];
                y[(((int64_t)b * Cout + co) * Ho + oh) * Wo + ow] = apply_act(acc, act);
            }
        }
    }
}

/*
 * Binary activations (Sec. 7 names tiled networks with binary weights AND binary activations as the
 * next step; Sec. 2 recalls that such networks, XNOR-Net among them, binarise the activations with
 * the sign function and keep a real scaling factor).  The paper fixes no formula for this case; the
 * reading taken here, listed in the design notes, is the smallest extension of Sec. 3:
 *   a[t][j]  = +1 if x[t][j] > 0 else -1            (the threshold rule of Eq. 3, applied to x)
 *   beta[t]  = ||x[t][:]||_1 / n                     (the scaling of Eq. 6, applied to one input row)
 *   y[t][i]  = act( beta[t] * sum_j B_hat[i][j] * a[t][j] + bias[i] )
 * with B_hat the scaled tiled weight of Eq. 4-8.  Everything below is that definition written out.
 */

/* Threshold + row scale of one activation matrix.  bits[t*n + j] in {0,1}; beta nullable. */
void tbn_oracle_binarize(const double *x, int64_t T, int32_t n, uint8_t *bits, float *beta)
{
    for (int64_t t = 0; t < T; ++t) {
        double a = 0.0;
        for (int32_t j = 0; j < n; ++j) {
            const double v = x[t * n + j];
            bits[t * n + j] = (v > 0.0) ? 1 : 0;           /* zero, negative zero and NaN give -1 */
            a += fabs(v);
        }
        if (beta) beta[t] = (float)(a / (double)n);
    }
}

/*
 * The integer part of the binary-activation layer: D[t][i] = sum_j b[i][j] * a[t][j] with
 * b[i][j] = +-1 the unscaled tiled weight (Eq. 4-5: bit (i*n + j) mod q of the tile) and a = +-1.
 * Exact in integers.  abits: T x n values in {0,1}.
 */
void tbn_oracle_linear_bin_int(const uint8_t *abits, int64_t T, int32_t n, int32_t m,
                               const uint32_t *words, int64_t q, int64_t *D)
{
    const int64_t total = T * (int64_t)m;
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < total; ++o) {
        const int64_t t = o / m;
        const int32_t i = (int32_t)(o % m);
        int64_t acc = 0;
        for (int32_t j = 0; j < n; ++j) {
            const int64_t f = ((int64_t)i * n + j) % q;
            const int b = ((words[f >> 5] >> (f & 31)) & 1u) ? 1 : -1;
            const int a = abits[t * n + j] ? 1 : -1;
            acc += b * a;
        }
        D[o] = acc;
    }
}
