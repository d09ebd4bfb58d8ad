/*
 * LoRDBA adapter-forward ORACLE -- test infrastructure, not product code.
 *
 * A plain, slow, float64 CPU statement of what the unmerged double-binary
 * adapter branch computes.  Only the tests, the smoke check and the bench's
 * CPU-baseline leg may call it; the CUDA library neither includes nor links
 * anything from this directory, and this file includes nothing of the CUDA
 * library.
 *
 * Notation (paper Def. 1 -> this file):
 *   N, M            -> d_in, d_out        R -> r
 *   B1 (N x R)      -> A_sign = B1^T  (r x d_in,  int8 +-1, row-major)
 *   B2 (R x M)      -> B_sign = B2^T  (d_out x r, int8 +-1, row-major)
 *   alpha, beta, gamma -> s_in (d_in), s_r (r), s_out (d_out)
 *   X (T x N)       -> x, row-major, one token per row
 *
 * Pins (all in tests/, run without a GPU):
 *   oracle_adapter_forward      : dense Delta-W matmul (Eq. 4), exhaustive
 *                                 tiny sign matrices, all-(+1) closed form,
 *                                 linearity, gauge and zero-padding
 *                                 invariants, rank bound.
 *   oracle_adapter_forward_ell  : same, plus "extra zero envelope is a no-op".
 *   oracle_pack_* / unpack_*    : hand-written words, exhaustive round trip,
 *                                 popcount, zero pad bits.
 *   oracle_adapter_bits, _bpw_tot, _bandwidth_ratio : the sizes and ratios
 *                                 the paper prints (tests/golden/).
 * No function here is "parity unpinned".
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Number of threads the token loop will use (1 without OpenMP). */
int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* sign(0) = +1 (paper, Notation paragraph): negative -> -1, everything else -> +1. */
static int sgn_of(int8_t v) { return v < 0 ? -1 : +1; }

/*
 * Sign accumulation, Eq. 9: the sum of the entries whose sign is +1 minus the
 * sum of the entries whose sign is -1.  No multiplication by the sign.
 */
static double sign_accumulate(const double *w, const int8_t *sgn, int64_t n)
{
    double plus = 0.0, minus = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (sgn_of(sgn[i]) > 0) plus += w[i];
        else                    minus += w[i];
    }
    return plus - minus;
}

/*
 * One token through the evaluation order of Eq. 8,
 *   ((((x D_alpha) B1) D_beta) B2) D_gamma,
 * added to the row of y that already holds the base projection (Def. 1:
 * y = W0^T x + Delta-W^T x).  xs (d_in) and z (r) are caller scratch.
 */
static void forward_token(const double *x, const int8_t *A_sign, const int8_t *B_sign,
                          const double *s_in, const double *s_r, const double *s_out,
                          double *y, int64_t d_in, int64_t d_out, int64_t r,
                          double *xs, double *z)
{
    for (int64_t i = 0; i < d_in; ++i) xs[i] = x[i] * s_in[i];           /* x D_alpha   */
    for (int64_t k = 0; k < r; ++k) {
        double u = sign_accumulate(xs, A_sign + k * d_in, d_in);         /* (.) B1      */
        z[k] = u * s_r[k];                                               /* (.) D_beta  */
    }
    for (int64_t j = 0; j < d_out; ++j) {
        double v = sign_accumulate(z, B_sign + j * r, r);                /* (.) B2      */
        y[j] += v * s_out[j];                                            /* (.) D_gamma, += */
    }
}

/*
 * y[t,:] += adapter(x[t,:]) for t < T, canonical single envelope (Eq. 8).
 * x: T x d_in with row pitch ldx, y: T x d_out with row pitch ldy (elements).
 * Returns 0, or -1 on bad sizes / allocation failure.
 */
int oracle_adapter_forward(const double *x, const int8_t *A_sign, const int8_t *B_sign,
                           const double *s_in, const double *s_r, const double *s_out,
                           double *y, int64_t T, int64_t d_in, int64_t d_out, int64_t r,
                           int64_t ldx, int64_t ldy)
{
    if (T < 0 || d_in < 0 || d_out < 0 || r < 0 || ldx < d_in || ldy < d_out) return -1;
    int failed = 0;
#pragma omp parallel
    {
        double *xs = (double *)malloc(sizeof(double) * (size_t)(d_in > 0 ? d_in : 1));
        double *z  = (double *)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
        if (!xs || !z) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(static)
            for (int64_t t = 0; t < T; ++t)
                forward_token(x + t * ldx, A_sign, B_sign, s_in, s_r, s_out,
                              y + t * ldy, d_in, d_out, r, xs, z);
        }
        free(xs);
        free(z);
    }
    return failed ? -1 : 0;
}

/*
 * Multi-envelope adapter (Eq. 4 with ell >= 1): the sum of ell terms that
 * share the two sign carriers; envelope e has scales s_in[e,:], s_r[e,:],
 * s_out[e,:] (row-major ell x d_in, ell x r, ell x d_out).
 */
int oracle_adapter_forward_ell(const double *x, const int8_t *A_sign, const int8_t *B_sign,
                               const double *s_in, const double *s_r, const double *s_out,
                               double *y, int64_t T, int64_t d_in, int64_t d_out, int64_t r,
                               int64_t ell, int64_t ldx, int64_t ldy)
{
    if (ell < 0) return -1;
    for (int64_t e = 0; e < ell; ++e) {
        int rc = oracle_adapter_forward(x, A_sign, B_sign, s_in + e * d_in, s_r + e * r,
                                        s_out + e * d_out, y, T, d_in, d_out, r, ldx, ldy);
        if (rc) return rc;
    }
    return 0;
}

/* ------------------------------------------------------------------------
 * Bit-packed carriers.  The paper only says the carriers are bit-packed; the
 * layout below is this library's, written down once here in integer loops.
 *
 *  A carrier (A_sign, r x d_in): the columns are cut into blocks of 64; block
 *    b holds r consecutive 64-bit groups, one per row k, each stored as two
 *    32-bit words (low word first).  Column i of row k is bit (i mod 32) of
 *    word ((i/64)*r + k)*2 + (i mod 64)/32; ceil(d_in/64)*r*2 words.
 *  B carrier (B_sign, d_out x r): one dense little-endian bit stream of the
 *    row-major matrix: entry (j,k) is bit b = j*r + k, i.e. bit (b mod 32) of
 *    word b/32; ceil(d_out*r/32) words.
 *  Bit 1 <=> +1, bit 0 <=> -1.  Pad bits are 0.
 * ------------------------------------------------------------------------ */

int64_t oracle_packed_words(int64_t rows, int64_t cols, int role)
{
    if (rows < 0 || cols < 0) return -1;
    if (role == 0) return ((cols + 63) / 64) * rows * 2;
    if (role == 1) return (rows * cols + 31) / 32;
    return -1;
}

int oracle_pack_signs(const int8_t *signs, int64_t rows, int64_t cols, int role, uint32_t *packed)
{
    int64_t nw = oracle_packed_words(rows, cols, role);
    if (nw < 0) return -1;
    for (int64_t w = 0; w < nw; ++w) packed[w] = 0u;
    for (int64_t a = 0; a < rows; ++a) {
        for (int64_t b = 0; b < cols; ++b) {
            if (sgn_of(signs[a * cols + b]) < 0) continue;
            int64_t word, bit;
            if (role == 0) { word = ((b / 64) * rows + a) * 2 + (b % 64) / 32; bit = b % 32; }
            else           { int64_t s = a * cols + b; word = s / 32; bit = s % 32; }
            packed[word] |= (uint32_t)1u << bit;
        }
    }
    return 0;
}

int oracle_unpack_signs(const uint32_t *packed, int64_t rows, int64_t cols, int role, int8_t *signs)
{
    if (oracle_packed_words(rows, cols, role) < 0) return -1;
    for (int64_t a = 0; a < rows; ++a) {
        for (int64_t b = 0; b < cols; ++b) {
            int64_t word, bit;
            if (role == 0) { word = ((b / 64) * rows + a) * 2 + (b % 64) / 32; bit = b % 32; }
            else           { int64_t s = a * cols + b; word = s / 32; bit = s % 32; }
            signs[a * cols + b] = ((packed[word] >> bit) & 1u) ? (int8_t)1 : (int8_t)-1;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------
 * Storage formulas.
 * ------------------------------------------------------------------------ */

/* Eq. 5: bits(theta) = R(N+M) + 16 ell (N+R+M). */
int64_t oracle_adapter_bits(int64_t d_in, int64_t d_out, int64_t r, int64_t ell)
{
    return r * (d_in + d_out) + 16 * ell * (d_in + r + d_out);
}

/* Bits of an fp16 LoRA of rank r0 (Preliminaries): 16 r0 (N+M). */
int64_t oracle_lora_fp16_bits(int64_t d_in, int64_t d_out, int64_t r0)
{
    return 16 * r0 * (d_in + d_out);
}

/* Eq. 6: BPW_tot = bits(theta) / (r0 (N+M)). */
double oracle_bpw_tot(int64_t d_in, int64_t d_out, int64_t r, int64_t ell, int64_t r0)
{
    return (double)oracle_adapter_bits(d_in, d_out, r, ell) / (double)(r0 * (d_in + d_out));
}

/* Adapter-bandwidth ratio at ell = 1, R = r0 (Section 5.2, Analysis). */
double oracle_bandwidth_ratio(int64_t d_in, int64_t d_out, int64_t r0)
{
    return (double)oracle_lora_fp16_bits(d_in, d_out, r0) /
           (double)oracle_adapter_bits(d_in, d_out, r0, 1);
}
