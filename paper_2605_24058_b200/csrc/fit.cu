// Closed-form scale updates of the adapter fit (Appendix "Closed-form scale updates for
// PTQ-LoRDBA"): one block-coordinate sweep alpha -> beta -> gamma of
//
//     min  1/2 || T - diag(alpha) B1 diag(beta) B2 diag(gamma) ||_F^2        (Eq. scale-joint)
//
// with the bit-packed carriers fixed.  In the library's orientation T is d_in x d_out,
// B1 = A_sign^T, B2 = B_sign^T, (alpha, beta, gamma) = (s_in, s_r, s_out).
//
// Nothing of size d_in x d_out is ever formed besides the target itself.  The two products that
// touch T are the sign accumulations of the forward pass and of its adjoint, applied to T:
//
//     W[i,k] = sum_j T[i,j] gamma_j B_sign[j,k]          (rows of T through B2^T diag(gamma))
//     V[k,j] = sum_i alpha_i A_sign[k,i] T[i,j]          (columns of T through diag(alpha) B1)
//
// and every update follows from them and from two r x r Gram matrices,
// Gq = Q Q^T (Q = B2 diag(gamma)) and Gp = P^T P (P = diag(alpha) B1):
//
//     alpha_i = <c_i, W[i,:]> / (c_i^T Gq c_i),   c_i = B1[i,:] * beta      (Eq. alpha-update)
//     beta    = ((Gp o Gq))^+ h,   h_k = sum_i alpha_i B1[i,k] W[i,k]      (Eq. beta-gram, beta-pinv)
//     gamma_j = <d_j, V[:,j]> / (d_j^T Gp d_j),   d_j = beta * B2[:,j]      (Eq. gamma-update)
//
// (a zero denominator gives 0, the minimum-norm solution).  The passes over T are float32 FMAs
// against signed scales expanded once per chunk into shared memory (per-lane or per-thread runs,
// then a tree or a fixed-order sum); everything of size r x r, the quotients and the
// pseudo-inverse (cyclic Jacobi eigendecomposition, eigenvalues below r eps lambda_max dropped)
// are float64.  All reductions run in a fixed order: results are deterministic.
#include <cstring>

#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kFitThreads = 256;
constexpr int kColsPerBlock = 128;      // columns of T per CTA of the column pass
constexpr int kMaxRowChunks = 16;       // partial sums of the column pass
constexpr int kParts = 8;               // partial sums of the Gram matrices and of h (added in a fixed order by their readers)

// r sign bits of row j of B_sign (role-1 stream: bit j*r + k), bit 1 = +1
__device__ __forceinline__ uint64_t b_bits(const uint32_t *__restrict__ pb, int64_t n_words, int64_t j, int r)
{
    const int64_t bit = j * r;
    const int64_t w = bit >> 5;
    const int sh = (int)(bit & 31);
    uint64_t lo = __ldg(pb + w);
    uint64_t mid = (w + 1 < n_words) ? __ldg(pb + w + 1) : 0u;
    uint64_t v = (lo | (mid << 32)) >> sh;
    if (sh > 0 && r > 64 - sh) {
        const uint64_t hi = (w + 2 < n_words) ? __ldg(pb + w + 2) : 0u;
        v |= hi << (64 - sh);
    }
    return r >= 64 ? v : (v & ((1ull << r) - 1ull));
}

// r sign bits of column i of A_sign (role-0 blocks: entry (k,i) is bit i%32 of word ((i/64) r + k) 2 + (i%64)/32)
__device__ __forceinline__ uint64_t a_bits(const uint32_t *__restrict__ pa, int64_t i, int r)
{
    const uint32_t *blk = pa + (i >> 6) * (int64_t)r * 2 + ((i & 63) >> 5);
    const int b = (int)(i & 31);
    // eight independent loads at a time: the r words are far apart in time only if they wait for
    // one another
    uint64_t v = 0;
    for (int k0 = 0; k0 < r; k0 += 8) {
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = (k0 + i < r) ? __ldg(blk + 2 * (k0 + i)) : 0u;
#pragma unroll
        for (int i = 0; i < 8; ++i) v |= (uint64_t)((w[i] >> b) & 1u) << (k0 + i);
    }
    return v;
}

// ---- W[i,k] = sum_j T[i,j] gamma_j B_sign[j,k] ----------------------------------------------
// A CTA owns 8 * RB rows of T (a warp RB of them) and walks the columns 128 at a time: the chunk's
// signed scales gamma_j B_sign[j,k] are expanded once into shared memory and serve every row; a
// lane takes four consecutive columns (one 16-byte load per row when the rows allow it) and keeps
// RB x RP partial sums, joined by a shuffle tree at the end (fixed order).
constexpr int kRowCols = 128;

template <int RP, int RB>
__global__ void __launch_bounds__(kFitThreads)
fit_row_pass_kernel(const float *__restrict__ T, int64_t ld, const uint32_t *__restrict__ pb,
                    const float *__restrict__ gamma, int64_t d_in, int64_t d_out, int r, int vec4,
                    float *__restrict__ W)
{
    constexpr int kStride = RP + 4;                    // floats per column: 16-byte reads without bank conflicts
    // column c of the chunk sits at slot (c % 4) * 32 + c / 4, so that the four columns of lane l are
    // the slots l, 32 + l, 64 + l, 96 + l: consecutive lanes read consecutive slots
    __shared__ __align__(16) float S[kRowCols * kStride];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row0 = ((int64_t)blockIdx.x * (kFitThreads / 32) + warp) * RB;
    const int64_t n_words = (d_out * r + 31) / 32;
    float acc[RB][RP];
#pragma unroll
    for (int b = 0; b < RB; ++b)
#pragma unroll
        for (int k = 0; k < RP; ++k) acc[b][k] = 0.0f;
    for (int64_t j0 = 0; j0 < d_out; j0 += kRowCols) {
        // this chunk's rows of T first: the loads fly while the signs are expanded
        float t[RB][4];
        const int64_t jl = j0 + 4 * lane;
#pragma unroll
        for (int b = 0; b < RB; ++b) {
            const bool row_ok = row0 + b < d_in;
            if (vec4 && row_ok && jl + 4 <= d_out) {
                const float4 v = __ldcs(reinterpret_cast<const float4 *>(T + (row0 + b) * ld + jl));
                t[b][0] = v.x; t[b][1] = v.y; t[b][2] = v.z; t[b][3] = v.w;
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) t[b][i] = (row_ok && jl + i < d_out) ? T[(row0 + b) * ld + jl + i] : 0.0f;
            }
        }
        __syncthreads();
        if (threadIdx.x < kRowCols) {
            const int c = threadIdx.x;
            const int64_t j = j0 + c;
            const bool in = j < d_out;
            const uint64_t bits = in ? b_bits(pb, n_words, j, r) : 0ull;
            const float g = in ? __ldg(gamma + j) : 0.0f;
            float *dst = S + ((c & 3) * 32 + (c >> 2)) * kStride;
#pragma unroll
            for (int k = 0; k < RP; ++k) dst[k] = (k < r) ? (((bits >> k) & 1ull) ? g : -g) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float *src = S + (i * 32 + lane) * kStride;
#pragma unroll
            for (int k4 = 0; k4 < RP / 4; ++k4) {
                const float4 sv = *reinterpret_cast<const float4 *>(src + 4 * k4);
#pragma unroll
                for (int b = 0; b < RB; ++b) {
                    acc[b][4 * k4] = fmaf(t[b][i], sv.x, acc[b][4 * k4]);
                    acc[b][4 * k4 + 1] = fmaf(t[b][i], sv.y, acc[b][4 * k4 + 1]);
                    acc[b][4 * k4 + 2] = fmaf(t[b][i], sv.z, acc[b][4 * k4 + 2]);
                    acc[b][4 * k4 + 3] = fmaf(t[b][i], sv.w, acc[b][4 * k4 + 3]);
                }
            }
        }
    }
#pragma unroll
    for (int b = 0; b < RB; ++b)
#pragma unroll
        for (int k = 0; k < RP; ++k) {
            float v = acc[b][k];
#pragma unroll
            for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
            if (lane == 0 && k < r && row0 + b < d_in) W[(row0 + b) * r + k] = v;
        }
}

// ---- V[c][k][j] = sum over the rows i of chunk c of alpha_i A_sign[k,i] T[i,j] ---------------
// A thread owns one column of T; the signed scales alpha_i A_sign[k,i] of 64 rows at a time (one
// block of the A carrier) are expanded once into shared memory and read by every thread at the
// same address (a broadcast).
template <int RP>
__global__ void __launch_bounds__(kColsPerBlock)
fit_col_pass_kernel(const float *__restrict__ T, int64_t ld, const uint32_t *__restrict__ pa,
                    const float *__restrict__ alpha, int64_t d_in, int64_t d_out, int r, int64_t rows_per_chunk,
                    float *__restrict__ Vpart)
{
    __shared__ __align__(16) float S[64 * RP];
    const int64_t j = (int64_t)blockIdx.x * kColsPerBlock + threadIdx.x;
    const int64_t i_begin = (int64_t)blockIdx.y * rows_per_chunk;
    const int64_t i_end = (i_begin + rows_per_chunk < d_in) ? i_begin + rows_per_chunk : d_in;
    float acc[RP];
#pragma unroll
    for (int k = 0; k < RP; ++k) acc[k] = 0.0f;
    for (int64_t i0 = i_begin; i0 < i_end; i0 += 64) {         // one 64-column block of the A carrier
        __syncthreads();
        if (threadIdx.x < 64) {
            const int64_t i = i0 + threadIdx.x;
            const bool in = i < i_end;
            const uint64_t bits = in ? a_bits(pa, i, r) : 0ull;
            const float a = in ? __ldg(alpha + i) : 0.0f;
#pragma unroll
            for (int k = 0; k < RP; ++k) S[threadIdx.x * RP + k] = (k < r) ? (((bits >> k) & 1ull) ? a : -a) : 0.0f;
        }
        __syncthreads();
        const int n = (int)((i_end - i0 < 64) ? (i_end - i0) : 64);
        if (j < d_out) {
#pragma unroll 16
            for (int il = 0; il < n; ++il) {
                const float t = __ldcs(T + (i0 + il) * ld + j);
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4) {
                    const float4 sv = *reinterpret_cast<const float4 *>(&S[il * RP + 4 * k4]);
                    acc[4 * k4] = fmaf(t, sv.x, acc[4 * k4]);
                    acc[4 * k4 + 1] = fmaf(t, sv.y, acc[4 * k4 + 1]);
                    acc[4 * k4 + 2] = fmaf(t, sv.z, acc[4 * k4 + 2]);
                    acc[4 * k4 + 3] = fmaf(t, sv.w, acc[4 * k4 + 3]);
                }
            }
        }
    }
    if (j < d_out) {
#pragma unroll
        for (int k = 0; k < RP; ++k)
            if (k < r) Vpart[((int64_t)blockIdx.y * r + k) * d_out + j] = acc[k];
    }
}

// ---- G[k][l] = sum_n s_n^2 B[n,k] B[n,l] over one carrier (float64), one CTA per row k --------
template <int ROLE>
__global__ void __launch_bounds__(kFitThreads)
fit_gram_kernel(const uint32_t *__restrict__ packed, const float *__restrict__ scale, int64_t n, int r,
                int64_t n_words, double *__restrict__ G)
{
    __shared__ double red[kFitThreads / 32][64];
    const int k = blockIdx.x;
    const int64_t per = (n + kParts - 1) / kParts;
    const int64_t e_begin = (int64_t)blockIdx.y * per, e_end = (e_begin + per < n) ? e_begin + per : n;
    double acc[64];
#pragma unroll
    for (int l = 0; l < 64; ++l) acc[l] = 0.0;
    for (int64_t e = e_begin + threadIdx.x; e < e_end; e += kFitThreads) {
        const double s = (double)__ldg(scale + e);
        const double s2 = s * s;
        const uint64_t bits = (ROLE == 1) ? b_bits(packed, n_words, e, r) : a_bits(packed, e, r);
        // B[e,k] B[e,l] = +1 where the two bits agree
        const uint64_t agree = ~(bits ^ (((bits >> k) & 1ull) ? ~0ull : 0ull));
#pragma unroll
        for (int l = 0; l < 64; ++l) acc[l] += ((agree >> l) & 1ull) ? s2 : -s2;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int l = 0; l < 64; ++l) {
        double v = acc[l];
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
        if (lane == 0) red[warp][l] = v;
    }
    __syncthreads();
    if (threadIdx.x < r) {
        double v = 0.0;
        for (int w = 0; w < kFitThreads / 32; ++w) v += red[w][threadIdx.x];
        G[((int64_t)blockIdx.y * r + k) * r + threadIdx.x] = v;       // part blockIdx.y
    }
}

// sum of the kParts partial r x r matrices (or r-vectors), in a fixed order
__device__ __forceinline__ double sum_parts(const double *__restrict__ parts, int stride, int e)
{
    double v = 0.0;
#pragma unroll
    for (int p = 0; p < kParts; ++p) v += parts[(int64_t)p * stride + e];
    return v;
}

// ---- alpha_i = <c_i, W[i,:]> / (c_i^T Gq c_i), c_i = B1[i,:] * beta (Eq. alpha-update) ---------
__global__ void __launch_bounds__(kFitThreads)
fit_alpha_kernel(const uint32_t *__restrict__ pa, const float *__restrict__ W, const double *__restrict__ Gq,
                 const float *__restrict__ beta, int64_t d_in, int r, float *__restrict__ alpha)
{
    __shared__ double g[64 * 64];
    __shared__ double b[64];
    for (int e = threadIdx.x; e < r * r; e += kFitThreads) g[e] = sum_parts(Gq, r * r, e);
    if (threadIdx.x < r) b[threadIdx.x] = (double)beta[threadIdx.x];
    __syncthreads();
    const int64_t i = (int64_t)blockIdx.x * kFitThreads + threadIdx.x;
    if (i >= d_in) return;
    const uint64_t bits = a_bits(pa, i, r);
    double num = 0.0, den = 0.0;
    for (int k = 0; k < r; ++k) {
        const double ck = ((bits >> k) & 1ull) ? b[k] : -b[k];
        num += ck * (double)W[i * r + k];
        double row = 0.0;
        for (int l = 0; l < r; ++l) row += g[k * r + l] * (((bits >> l) & 1ull) ? b[l] : -b[l]);
        den += ck * row;
    }
    alpha[i] = den > 0.0 ? (float)(num / den) : 0.0f;
}

// ---- gamma_j = <d_j, V[:,j]> / (d_j^T Gp d_j), d_j = beta * B2[:,j] (Eq. gamma-update) ---------
__global__ void __launch_bounds__(kFitThreads)
fit_gamma_kernel(const uint32_t *__restrict__ pb, const float *__restrict__ Vpart, int chunks,
                 const double *__restrict__ Gp, const float *__restrict__ beta, int64_t d_out, int r,
                 float *__restrict__ gamma)
{
    __shared__ double g[64 * 64];
    __shared__ double b[64];
    for (int e = threadIdx.x; e < r * r; e += blockDim.x) g[e] = sum_parts(Gp, r * r, e);
    if (threadIdx.x < r) b[threadIdx.x] = (double)beta[threadIdx.x];
    __syncthreads();
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d_out) return;
    const uint64_t bits = b_bits(pb, (d_out * r + 31) / 32, j, r);
    double num = 0.0, den = 0.0;
    for (int k = 0; k < r; ++k) {
        double v = 0.0;
#pragma unroll 8
        for (int c = 0; c < chunks; ++c) v += (double)Vpart[((int64_t)c * r + k) * d_out + j];   // fixed order
        const double dk = ((bits >> k) & 1ull) ? b[k] : -b[k];
        num += dk * v;
        double row = 0.0;
        for (int l = 0; l < r; ++l) row += g[k * r + l] * (((bits >> l) & 1ull) ? b[l] : -b[l]);
        den += dk * row;
    }
    gamma[j] = den > 0.0 ? (float)(num / den) : 0.0f;
}

// ---- h_k = sum_i alpha_i B1[i,k] W[i,k] (Eq. beta-gram): kParts CTAs, fixed-order trees ------------
__global__ void __launch_bounds__(kFitThreads)
fit_h_kernel(const uint32_t *__restrict__ pa, const float *__restrict__ W, const float *__restrict__ alpha,
             int64_t d_in, int r, double *__restrict__ h)
{
    __shared__ double red[(kFitThreads / 32) * 64];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double acc[64];
#pragma unroll
    for (int k = 0; k < 64; ++k) acc[k] = 0.0;
    const int64_t per = (d_in + kParts - 1) / kParts;
    const int64_t i_begin = (int64_t)blockIdx.x * per, i_end = (i_begin + per < d_in) ? i_begin + per : d_in;
    for (int64_t i = i_begin + tid; i < i_end; i += kFitThreads) {
        const uint64_t bits = a_bits(pa, i, r);
        const double a = (double)alpha[i];
#pragma unroll
        for (int k = 0; k < 64; ++k)
            if (k < r) acc[k] += (((bits >> k) & 1ull) ? a : -a) * (double)W[i * r + k];
    }
#pragma unroll
    for (int k = 0; k < 64; ++k) {
        double v = acc[k];
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
        if (lane == 0) red[warp * 64 + k] = v;
    }
    __syncthreads();
    if (tid < r) {
        double v = 0.0;
        for (int w = 0; w < kFitThreads / 32; ++w) v += red[w * 64 + tid];
        h[blockIdx.x * r + tid] = v;            // part blockIdx.x
    }
}

// ---- beta = (Gp o Gq)^+ h (Eq. beta-Schur, Eq. beta-pinv): one CTA of 1024 threads ----------------
// Shared memory (dynamic): A and E, n rows of n + 1 doubles each (n = r rounded up to even), then the
// rotations of a round (2 x 64), h (64), the eigen-coefficients (64) and 2 x 32 partial norms.
constexpr int kBetaThreads = 1024;      // at most; small systems use fewer (a barrier of 128 threads is cheaper)

__global__ void __launch_bounds__(kBetaThreads)
fit_beta_kernel(const double *__restrict__ Gp, const double *__restrict__ Gq, const double *__restrict__ hvec, int r,
                float *__restrict__ beta)
{
    extern __shared__ double sh[];
    const int n = (r + 1) & ~1;
    const int ns = n + 1;        // padded row length: column walks without bank conflicts
    double *A = sh, *E = A + n * ns, *cs = E + n * ns, *h = cs + 2 * 64, *coef = h + 64, *part = coef + 64;
    __shared__ double off_norm, all_norm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x;

    for (int e = tid; e < n * n; e += nthr) {
        const int p = e / n, q = e - p * n;
        A[p * ns + q] = (p < r && q < r) ? sum_parts(Gp, r * r, p * r + q) * sum_parts(Gq, r * r, p * r + q) : 0.0;   // Eq. beta-Schur
        E[p * ns + q] = (p == q) ? 1.0 : 0.0;
    }
    if (tid < 64) h[tid] = (tid < r) ? sum_parts(hvec, r, tid) : 0.0;
    __syncthreads();

    // cyclic Jacobi, n / 2 disjoint rotations per round (round-robin pairing), at most 40 sweeps
    for (int sweep = 0; sweep < 40; ++sweep) {
        double off = 0.0, all = 0.0;
        for (int e = tid; e < n * n; e += nthr) {
            const int p = e / n, q = e - p * n;
            const double v = A[p * ns + q] * A[p * ns + q];
            all += v;
            if (p != q) off += v;
        }
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) {
            off += __shfl_xor_sync(0xffffffffu, off, s);
            all += __shfl_xor_sync(0xffffffffu, all, s);
        }
        if (lane == 0) { part[warp] = off; part[32 + warp] = all; }
        __syncthreads();
        if (tid == 0) {
            double o = 0.0, a = 0.0;
            for (int w = 0; w < nthr / 32; ++w) { o += part[w]; a += part[32 + w]; }
            off_norm = o;
            all_norm = a;
        }
        __syncthreads();
        // off-diagonal mass below 1e-12 of the whole (squares: 1e-24): the rotations left only move
        // rounding noise (they stall near n eps, which a tighter test would never see)
        if (off_norm <= 1e-24 * all_norm) break;
        for (int round = 0; round < n - 1; ++round) {
            // pair m of this round: (n-1, round) for m = 0, else ((round+m) % (n-1), (round-m) mod (n-1))
            if (tid < n / 2) {
                const int m = tid;
                const int p = (m == 0) ? n - 1 : (round + m) % (n - 1);
                const int q = (m == 0) ? round : (round - m + (n - 1)) % (n - 1);
                const double apq = A[p * ns + q];
                double c = 1.0, s = 0.0;
                if (apq != 0.0) {
                    const double theta = (A[q * ns + q] - A[p * ns + p]) / (2.0 * apq);
                    const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                    c = 1.0 / sqrt(t * t + 1.0);
                    s = t * c;
                }
                cs[2 * m] = c;
                cs[2 * m + 1] = s;
            }
            __syncthreads();
            // columns: A <- A J, E <- E J (task = row t, pair m)
            for (int task = tid; task < n * (n / 2); task += nthr) {
                const int t = task / (n / 2), m = task - t * (n / 2);
                const int p = (m == 0) ? n - 1 : (round + m) % (n - 1);
                const int q = (m == 0) ? round : (round - m + (n - 1)) % (n - 1);
                const double c = cs[2 * m], s = cs[2 * m + 1];
                const double ap = A[t * ns + p], aq = A[t * ns + q];
                A[t * ns + p] = c * ap - s * aq;
                A[t * ns + q] = s * ap + c * aq;
                const double ep = E[t * ns + p], eq = E[t * ns + q];
                E[t * ns + p] = c * ep - s * eq;
                E[t * ns + q] = s * ep + c * eq;
            }
            __syncthreads();
            // rows: A <- J^T A (task = column t, pair m)
            for (int task = tid; task < n * (n / 2); task += nthr) {
                const int t = task / (n / 2), m = task - t * (n / 2);
                const int p = (m == 0) ? n - 1 : (round + m) % (n - 1);
                const int q = (m == 0) ? round : (round - m + (n - 1)) % (n - 1);
                const double c = cs[2 * m], s = cs[2 * m + 1];
                const double ap = A[p * ns + t], aq = A[q * ns + t];
                A[p * ns + t] = c * ap - s * aq;
                A[q * ns + t] = s * ap + c * aq;
            }
            __syncthreads();
        }
    }
    __syncthreads();
    // beta = sum over eigenpairs with lambda > r eps lambda_max of (v^T h / lambda) v
    if (tid == 0) {
        double lmax = 0.0;
        for (int k = 0; k < n; ++k) lmax = fmax(lmax, A[k * ns + k]);
        off_norm = (double)r * 2.220446049250313e-16 * lmax;
    }
    __syncthreads();
    if (tid < n) {
        const double lam = A[tid * ns + tid];
        double dot = 0.0;
        for (int p = 0; p < r; ++p) dot += E[p * ns + tid] * h[p];
        coef[tid] = (lam > off_norm) ? dot / lam : 0.0;
    }
    __syncthreads();
    if (tid < r) {
        double v = 0.0;
        for (int k = 0; k < n; ++k) v += E[tid * ns + k] * coef[k];
        beta[tid] = (float)v;
    }
}

int padded_rank(int r) { return r <= 8 ? 8 : r <= 16 ? 16 : r <= 32 ? 32 : 64; }

struct FitWorkspace {
    float *W;          // d_in x r
    float *Vpart;      // chunks x r x d_out
    double *Gq, *Gp;   // kParts partial r x r matrices each
    double *h;         // kParts partial r-vectors
    int chunks;
    int64_t rows_per_chunk;
    size_t bytes;
};

FitWorkspace carve(void *base, int64_t d_in, int64_t d_out, int r)
{
    FitWorkspace w;
    const int64_t blocks = (d_in + 63) / 64;
    const int64_t per = (blocks + kMaxRowChunks - 1) / kMaxRowChunks;
    w.rows_per_chunk = per * 64;
    w.chunks = (int)((d_in + w.rows_per_chunk - 1) / w.rows_per_chunk);
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    size_t off = 0;
    char *p = static_cast<char *>(base);
    w.W = reinterpret_cast<float *>(p + off); off += up((size_t)d_in * r * 4);
    w.Vpart = reinterpret_cast<float *>(p + off); off += up((size_t)w.chunks * r * d_out * 4);
    w.Gq = reinterpret_cast<double *>(p + off); off += up((size_t)kParts * r * r * 8);
    w.Gp = reinterpret_cast<double *>(p + off); off += up((size_t)kParts * r * r * 8);
    w.h = reinterpret_cast<double *>(p + off); off += up((size_t)kParts * r * 8);
    w.bytes = off;
    return w;
}

size_t beta_smem(int r)
{
    const int n = (r + 1) & ~1;
    return sizeof(double) * (size_t)(2 * n * (n + 1) + 2 * 64 + 64 + 64 + 64);
}

template <int RP, int RB>
void launch_row(const float *T, int64_t ld, const uint32_t *pb, const float *gamma, int64_t d_in, int64_t d_out, int r,
                float *W, cudaStream_t s)
{
    const int rows_per_block = (kFitThreads / 32) * RB;
    const int vec4 = (reinterpret_cast<uintptr_t>(T) % 16 == 0 && ld % 4 == 0) ? 1 : 0;
    fit_row_pass_kernel<RP, RB><<<(unsigned)((d_in + rows_per_block - 1) / rows_per_block), kFitThreads, 0, s>>>(
        T, ld, pb, gamma, d_in, d_out, r, vec4, W);
}

template <int RP>
void launch_col(const float *T, int64_t ld, const uint32_t *pa, const float *alpha, int64_t d_in, int64_t d_out, int r,
                const FitWorkspace &w, cudaStream_t s)
{
    const dim3 grid((unsigned)((d_out + kColsPerBlock - 1) / kColsPerBlock), (unsigned)w.chunks, 1);
    fit_col_pass_kernel<RP><<<grid, kColsPerBlock, 0, s>>>(T, ld, pa, alpha, d_in, d_out, r, w.rows_per_chunk, w.Vpart);
}

}  // namespace

size_t fit_workspace_bytes(int64_t d_in, int64_t d_out, int r) { return carve(nullptr, d_in, d_out, r).bytes; }

int launch_fit_scales(const float *target, int64_t ld, const uint32_t *pa, const uint32_t *pb, float *s_in, float *s_r,
                      float *s_out, int64_t d_in, int64_t d_out, int r, int sweeps, int axes, void *workspace,
                      cudaStream_t stream)
{
    const FitWorkspace w = carve(workspace, d_in, d_out, r);
    const int rp = padded_rank(r);
    static cudaError_t attr_rc = cudaFuncSetAttribute(fit_beta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                      (int)beta_smem(kMaxRank));
    if (attr_rc != cudaSuccess) return LORDBA_ECUDA;
    const int64_t b_words = (d_out * r + 31) / 32;
    for (int sweep = 0; sweep < sweeps; ++sweep) {
        // rows of T through B2^T diag(gamma), and Q Q^T
        if (axes & (LORDBA_FIT_ALPHA | LORDBA_FIT_BETA)) {
            switch (rp) {
                case 8:  launch_row<8, 2>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
                case 16: launch_row<16, 2>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
                case 32: launch_row<32, 1>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
                default: launch_row<64, 1>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
            }
            fit_gram_kernel<1><<<dim3(r, kParts), kFitThreads, 0, stream>>>(pb, s_out, d_out, r, b_words, w.Gq);
            count_launch(2);
        }
        if (axes & LORDBA_FIT_ALPHA) {
            fit_alpha_kernel<<<(unsigned)((d_in + kFitThreads - 1) / kFitThreads), kFitThreads, 0, stream>>>(
                pa, w.W, w.Gq, s_r, d_in, r, s_in);
            count_launch();
        }
        if (axes & (LORDBA_FIT_BETA | LORDBA_FIT_GAMMA)) {
            fit_gram_kernel<0><<<dim3(r, kParts), kFitThreads, 0, stream>>>(pa, s_in, d_in, r, 0, w.Gp);
            count_launch();
        }
        if (axes & LORDBA_FIT_BETA) {
            fit_h_kernel<<<kParts, kFitThreads, 0, stream>>>(pa, w.W, s_in, d_in, r, w.h);
            const int n_even = (r + 1) & ~1;
            int beta_threads = 128;              // one task per thread and phase when it fits: n * n / 2 tasks
            while (beta_threads < n_even * n_even / 2 && beta_threads < kBetaThreads) beta_threads *= 2;
            fit_beta_kernel<<<1, beta_threads, beta_smem(r), stream>>>(w.Gp, w.Gq, w.h, r, s_r);
            count_launch(2);
        }
        if (axes & LORDBA_FIT_GAMMA) {
            switch (rp) {
                case 8:  launch_col<8>(target, ld, pa, s_in, d_in, d_out, r, w, stream); break;
                case 16: launch_col<16>(target, ld, pa, s_in, d_in, d_out, r, w, stream); break;
                case 32: launch_col<32>(target, ld, pa, s_in, d_in, d_out, r, w, stream); break;
                default: launch_col<64>(target, ld, pa, s_in, d_in, d_out, r, w, stream); break;
            }
            fit_gamma_kernel<<<(unsigned)((d_out + kFitThreads - 1) / kFitThreads), kFitThreads, 0, stream>>>(
                pb, w.Vpart, w.chunks, w.Gp, s_r, d_out, r, s_out);
            count_launch(2);
        }
        if (cudaGetLastError() != cudaSuccess) return LORDBA_ECUDA;
    }
    return LORDBA_OK;
}

}  // namespace lordba
