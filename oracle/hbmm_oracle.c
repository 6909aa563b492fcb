/*
 * CPU oracle for the Hadamard Binary Matrix Multiply (HBMM) of HadaNets.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * method computes, written from the paper's definitions; it is what the CUDA
 * library is checked against.  It shares no code, header, table or constant with
 * the CUDA path and must never be called from it.  Everything is computed in
 * double precision from the definition; there is no blocking, packing trick or
 * reordering (OpenMP splits the outermost row loop only, which changes no
 * result because every output element is produced by one thread in a fixed
 * k-ascending order).
 *
 * Notation follows the paper: an input tensor X (rows x K, row-major) becomes
 * X~ = delta (.) Sign(X), where delta holds the mean absolute value of each run
 * of beta consecutive elements of a row (Section 3, Eq. 1-4).
 *
 * Parity status of every function here: pinned (see tests/test_oracle_pins.py):
 * closed forms, exact rational brute force, the paper's bit-packing example,
 * the storage ratio of Table 2, special cases beta = 1 and beta = K.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Number of beta-groups of a row of length K: ceil(K / beta)  (Section 4.2, text before Eq. 7). */
static int64_t n_groups(int64_t K, int64_t beta) { return (K + beta - 1) / beta; }

/*
 * Hadamard binarization of a 2-D tensor, row-wise (Eq. 1-2 for weights after the
 * reshape to (filters, -1); Eq. 3-4 for activations).
 *   delta[r,g] = (1/|g|) * sum_{k in group g} |x[r,k]|,  group g = columns [g*beta, min((g+1)*beta, K))
 *   sign[r,k]  = +1 if x[r,k] >= 0 else -1
 * Readings: the sums of Eq. 1 / Eq. 3 run over the beta elements of the group
 * (the printed upper limit "beta" is taken as beta-1); a tail group shorter than
 * beta is averaged over its own length, which keeps delta the L2-optimal scale
 * of its segment (Section 3.1.2) and makes beta = K the XNOR-Net case for any K.
 * Sign(0) = Sign(-0) = +1 (decided by the comparison x >= 0).
 */
void oracle_quantize(const float *x, int64_t rows, int64_t K, int64_t ldx, int64_t beta,
                     double *delta, int8_t *sign)
{
    int64_t G = n_groups(K, beta);
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; r++) {
        for (int64_t g = 0; g < G; g++) {
            int64_t k0 = g * beta, k1 = k0 + beta;
            if (k1 > K) k1 = K;
            double s = 0.0;
            for (int64_t k = k0; k < k1; k++) s += fabs((double)x[r * ldx + k]);
            delta[r * G + g] = s / (double)(k1 - k0);
        }
        for (int64_t k = 0; k < K; k++) sign[r * K + k] = (x[r * ldx + k] >= 0.0f) ? 1 : -1;
    }
}

/*
 * Gradient through the Hadamard binarization X~ = delta (.) Sign(X) (Section 3.1.3, Eq. 6, with the
 * straight-through estimator of Eq. 5 for dSign/dx).  gy = dC/dX~ (incoming), gx = dC/dX (result).
 * For element i of group g (n_g elements, s = Sign(x)):
 *   gx[i] = (1/n_g) * s_i * sum_{j in g} gy[j] * s_j        (delta depends on every |x_j| of the group)
 *         + delta_g * gy[i] * [ |x_i| <= 1 ]                 (Eq. 5: the estimator passes |x| <= 1)
 * Readings: the printed sum runs j = beta*floor(i/beta) .. beta*(floor(i/beta)+1), one index too many,
 * as in Eq. 1 / Eq. 3: it is taken over the beta elements of the group; a tail group uses its own
 * length, as in oracle_quantize; the paper's "delta_{l,i}, the absolute value of the binarized weight"
 * is the group scale.  Taken in the paper's order: first the group sum, then the two terms.
 */
void oracle_binarize_backward(const float *x, const float *gy, int64_t rows, int64_t K, int64_t ldx,
                              int64_t ldg, int64_t beta, double *gx)
{
    int64_t G = n_groups(K, beta);
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; r++) {
        for (int64_t g = 0; g < G; g++) {
            int64_t k0 = g * beta, k1 = k0 + beta;
            if (k1 > K) k1 = K;
            double n = (double)(k1 - k0), abs_sum = 0.0, gs = 0.0;
            for (int64_t k = k0; k < k1; k++) {
                double v = (double)x[r * ldx + k];
                abs_sum += fabs(v);
                gs += (double)gy[r * ldg + k] * (v >= 0.0 ? 1.0 : -1.0);
            }
            double delta = abs_sum / n;
            for (int64_t k = k0; k < k1; k++) {
                double v = (double)x[r * ldx + k];
                double sgn = v >= 0.0 ? 1.0 : -1.0;
                double ste = fabs(v) <= 1.0 ? 1.0 : 0.0;
                gx[r * K + k] = sgn * gs / n + delta * (double)gy[r * ldg + k] * ste;
            }
        }
    }
}

/* Storage rounding of the "full precision" scale tensor: fp32 (the paper's 32-bit
 * full precision, Section 4.1) -- value after round-to-nearest-even to float. */
void oracle_round_f32(double *v, int64_t n)
{
    for (int64_t i = 0; i < n; i++) v[i] = (double)(float)v[i];
}

/* Storage rounding to bfloat16 (1 sign, 8 exponent, 7 mantissa bits), round to
 * nearest, ties to even, applied to the fp32-rounded scale.  Scales are finite
 * and non-negative here; the carry out of the mantissa into the exponent is the
 * correct behaviour for a round-up across a binade. */
void oracle_round_bf16(double *v, int64_t n)
{
    for (int64_t i = 0; i < n; i++) {
        float f = (float)v[i];
        uint32_t u;
        memcpy(&u, &f, 4);
        uint32_t lower = u & 0xFFFFu, upper = u >> 16;
        if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1u;
        u = upper << 16;
        memcpy(&f, &u, 4);
        v[i] = (double)f;
    }
}

/* Bit-packing of the binary tensor (Section 4): -1 -> bit 0, +1 -> bit 1, element k
 * of a row goes to bit (k mod 32) of word (k div 32), least significant bit first;
 * bits beyond K and words beyond ceil(K/32) are zero. */
void oracle_pack(const int8_t *sign, int64_t rows, int64_t K, int64_t ld_words, uint32_t *bits)
{
    for (int64_t r = 0; r < rows; r++) {
        for (int64_t w = 0; w < ld_words; w++) bits[r * ld_words + w] = 0u;
        for (int64_t k = 0; k < K; k++)
            if (sign[r * K + k] > 0) bits[r * ld_words + k / 32] |= (uint32_t)1 << (k % 32);
    }
}

void oracle_unpack(const uint32_t *bits, int64_t rows, int64_t K, int64_t ld_words, int8_t *sign)
{
    for (int64_t r = 0; r < rows; r++)
        for (int64_t k = 0; k < K; k++)
            sign[r * K + k] = ((bits[r * ld_words + k / 32] >> (k % 32)) & 1u) ? 1 : -1;
}

/* X~[r,k] = delta[r, floor(k/beta)] * sign[r,k]   (Eq. 2 / Eq. 4, the Hadamard product written out). */
void oracle_dequant(const double *delta, const int8_t *sign, int64_t rows, int64_t K, int64_t beta,
                    double *xt)
{
    int64_t G = n_groups(K, beta);
    #pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; r++)
        for (int64_t k = 0; k < K; k++)
            xt[r * K + k] = delta[r * G + k / beta] * (double)sign[r * K + k];
}

/* beta = 1 leaves a tensor at full precision (Section 3.1: first/last layers): X~ = X. */
void oracle_widen(const float *x, int64_t rows, int64_t K, int64_t ldx, double *xt)
{
    for (int64_t r = 0; r < rows; r++)
        for (int64_t k = 0; k < K; k++) xt[r * K + k] = (double)x[r * ldx + k];
}

/* C[m,n] = sum_k A~[m,k] * W~[n,k], k ascending, double.  This is the product the
 * xHBNN kernel of Eq. 7 regroups: Eq. 7's per-group term is the signed dot of the
 * group's +-1 vectors times the two group scales. */
void oracle_matmul_nt(const double *at, const double *wt, int64_t M, int64_t N, int64_t K, double *c)
{
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; m++)
        for (int64_t n = 0; n < N; n++) {
            double s = 0.0;
            for (int64_t k = 0; k < K; k++) s += at[m * K + k] * wt[n * K + k];
            c[m * N + n] = s;
        }
}

/* Segments of the K axis on which both operands have a constant scale: a new
 * segment starts wherever a beta_a-group or a beta_w-group starts (Section 4.2:
 * with beta_a <= beta_w the finer segmentation decides the work).  beta == 1
 * contributes no boundary of its own here only if the caller passes beta = K
 * for it; callers use this for packed operands (beta >= 2). */
int64_t oracle_num_segments(int64_t K, int64_t beta_a, int64_t beta_w)
{
    int64_t t = 0;
    for (int64_t k = 0; k < K; k++)
        if (k % beta_a == 0 || k % beta_w == 0) t++;
    return t;
}

/*
 * Integer partial sums of Eq. 7, from the +-1 values by multiply and add (no
 * popcount anywhere, so the identity dot = n - 2*popc(xor) is a real cross-check):
 *   D[m,n,t] = sum_{k in segment t} sA[m,k] * sW[n,k]
 * and, when absref != NULL and both scale tensors are given, the magnitude
 * reference used by the floating-point tolerance:
 *   absref[m,n] = sum_t | deltaA[m,ga(t)] * deltaW[n,gw(t)] * D[m,n,t] |.
 * d may be NULL when only absref is wanted.
 */
void oracle_partials(const int8_t *sa, const int8_t *sw, int64_t M, int64_t N, int64_t K,
                     int64_t beta_a, int64_t beta_w,
                     const double *delta_a, const double *delta_w,
                     int32_t *d, double *absref)
{
    int64_t T = oracle_num_segments(K, beta_a, beta_w);
    int64_t Ga = n_groups(K, beta_a), Gw = n_groups(K, beta_w);
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; m++)
        for (int64_t n = 0; n < N; n++) {
            double r = 0.0;
            int64_t t = -1;
            int32_t acc = 0;
            for (int64_t k = 0; k <= K; k++) {
                int boundary = (k == K) || (k % beta_a == 0) || (k % beta_w == 0);
                if (boundary && t >= 0) {
                    if (d) d[(m * N + n) * T + t] = acc;
                    if (absref) {
                        int64_t klast = k - 1;
                        r += fabs(delta_a[m * Ga + klast / beta_a] * delta_w[n * Gw + klast / beta_w] * (double)acc);
                    }
                }
                if (k == K) break;
                if (boundary) { t++; acc = 0; }
                acc += (int32_t)sa[m * K + k] * (int32_t)sw[n * K + k];
            }
            if (absref) absref[m * N + n] = r;
        }
}

/*
 * im2col of an NCHW activation tensor for a kh x kw convolution: row m = (b, yo, xo)
 * (xo fastest), column k = (c, i, j) with c slowest -- the order Reshape(W, (S[0], -1))
 * gives a (filters, c, kh, kw) weight tensor (Algorithm 1; Section 3.1.1), so that
 * column k of the activation matrix meets column k of W^f.  Out-of-image taps are 0.
 */
void oracle_im2col(const float *x, int64_t B, int64_t C, int64_t H, int64_t W,
                   int64_t kh, int64_t kw, int64_t sh, int64_t sw, int64_t ph, int64_t pw,
                   float *out)
{
    int64_t Ho = (H + 2 * ph - kh) / sh + 1, Wo = (W + 2 * pw - kw) / sw + 1;
    int64_t K = C * kh * kw;
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < B * Ho * Wo; m++) {
        int64_t b = m / (Ho * Wo), yo = (m / Wo) % Ho, xo = m % Wo;
        for (int64_t c = 0; c < C; c++)
            for (int64_t i = 0; i < kh; i++)
                for (int64_t j = 0; j < kw; j++) {
                    int64_t y = yo * sh + i - ph, xx = xo * sw + j - pw;
                    float v = 0.0f;
                    if (y >= 0 && y < H && xx >= 0 && xx < W) v = x[((b * C + c) * H + y) * W + xx];
                    out[m * K + (c * kh + i) * kw + j] = v;
                }
    }
}
