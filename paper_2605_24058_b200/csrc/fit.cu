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
// (a zero denominator gives 0, the minimum-norm solution).  The passes over T accumulate in
// float32 (short per-lane runs, then a tree); everything of size r x r, the quotients and the
// pseudo-inverse (cyclic Jacobi eigendecomposition, eigenvalues below r eps lambda_max dropped)
// are float64.  All reductions run in a fixed order: results are deterministic.
#include <cstring>

#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kFitThreads = 256;
constexpr int kColsPerBlock = 128;      // columns of T per CTA of the column pass
constexpr int kMaxRowChunks = 16;       // partial sums of the column pass

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
    uint64_t v = 0;
    for (int k = 0; k < r; ++k) v |= (uint64_t)((__ldg(blk + 2 * k) >> b) & 1u) << k;
    return v;
}

__device__ __forceinline__ float signed_f(float v, uint64_t bits, int k)
{
    // +v when bit k is set, -v otherwise
    return __uint_as_float(__float_as_uint(v) ^ ((uint32_t)(~(bits >> k) & 1ull) << 31));
}

// ---- W[i,k] = sum_j T[i,j] gamma_j B_sign[j,k]: one warp per row of T ------------------------
template <int RP>
__global__ void __launch_bounds__(kFitThreads)
fit_row_pass_kernel(const float *__restrict__ T, int64_t ld, const uint32_t *__restrict__ pb,
                    const float *__restrict__ gamma, int64_t d_in, int64_t d_out, int r, float *__restrict__ W)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (kFitThreads / 32) + (threadIdx.x >> 5);
    if (row >= d_in) return;
    const int64_t n_words = (d_out * r + 31) / 32;
    float acc[RP];
#pragma unroll
    for (int k = 0; k < RP; ++k) acc[k] = 0.0f;
    const float *trow = T + row * ld;
    for (int64_t j = lane; j < d_out; j += 32) {
        const float t = trow[j] * __ldg(gamma + j);
        const uint64_t bits = b_bits(pb, n_words, j, r);
#pragma unroll
        for (int k = 0; k < RP; ++k) acc[k] += signed_f(t, bits, k);      // ranks >= r: unused
    }
#pragma unroll
    for (int k = 0; k < RP; ++k) {
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], s);
    }
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < RP; ++k)
            if (k < r) W[row * r + k] = acc[k];
    }
}

// ---- V[c][k][j] = sum over the rows i of chunk c of alpha_i A_sign[k,i] T[i,j] ---------------
template <int RP>
__global__ void __launch_bounds__(kColsPerBlock)
fit_col_pass_kernel(const float *__restrict__ T, int64_t ld, const uint32_t *__restrict__ pa,
                    const float *__restrict__ alpha, int64_t d_in, int64_t d_out, int r, int64_t rows_per_chunk,
                    float *__restrict__ Vpart)
{
    __shared__ uint64_t rowbits[64];
    __shared__ float arow[64];
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
            rowbits[threadIdx.x] = (i < i_end) ? a_bits(pa, i, r) : 0ull;
            arow[threadIdx.x] = (i < i_end) ? __ldg(alpha + i) : 0.0f;
        }
        __syncthreads();
        const int n = (int)((i_end - i0 < 64) ? (i_end - i0) : 64);
        if (j < d_out) {
            for (int il = 0; il < n; ++il) {
                const float t = T[(i0 + il) * ld + j] * arow[il];
                const uint64_t bits = rowbits[il];
#pragma unroll
                for (int k = 0; k < RP; ++k) acc[k] += signed_f(t, bits, k);
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
    double acc[64];
#pragma unroll
    for (int l = 0; l < 64; ++l) acc[l] = 0.0;
    for (int64_t e = threadIdx.x; e < n; e += kFitThreads) {
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
        G[k * r + threadIdx.x] = v;
    }
}

// ---- alpha_i = <c_i, W[i,:]> / (c_i^T Gq c_i), c_i = B1[i,:] * beta (Eq. alpha-update) ---------
__global__ void __launch_bounds__(kFitThreads)
fit_alpha_kernel(const uint32_t *__restrict__ pa, const float *__restrict__ W, const double *__restrict__ Gq,
                 const float *__restrict__ beta, int64_t d_in, int r, float *__restrict__ alpha)
{
    __shared__ double g[64 * 64];
    __shared__ double b[64];
    for (int e = threadIdx.x; e < r * r; e += kFitThreads) g[e] = Gq[e];
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
    for (int e = threadIdx.x; e < r * r; e += kFitThreads) g[e] = Gp[e];
    if (threadIdx.x < r) b[threadIdx.x] = (double)beta[threadIdx.x];
    __syncthreads();
    const int64_t j = (int64_t)blockIdx.x * kFitThreads + threadIdx.x;
    if (j >= d_out) return;
    const uint64_t bits = b_bits(pb, (d_out * r + 31) / 32, j, r);
    double num = 0.0, den = 0.0;
    for (int k = 0; k < r; ++k) {
        double v = 0.0;
        for (int c = 0; c < chunks; ++c) v += (double)Vpart[((int64_t)c * r + k) * d_out + j];   // fixed order
        const double dk = ((bits >> k) & 1ull) ? b[k] : -b[k];
        num += dk * v;
        double row = 0.0;
        for (int l = 0; l < r; ++l) row += g[k * r + l] * (((bits >> l) & 1ull) ? b[l] : -b[l]);
        den += dk * row;
    }
    gamma[j] = den > 0.0 ? (float)(num / den) : 0.0f;
}

// ---- beta = (Gp o Gq)^+ h, h_k = sum_i alpha_i B1[i,k] W[i,k] (Eq. beta-gram, Eq. beta-pinv): one CTA
// Shared memory (dynamic): A and E, n x n doubles each (n = r rounded up to even), then
// cs (n doubles), h (64), partial sums (threads / 32 x 64), eigen-coefficients (64).
__global__ void __launch_bounds__(kFitThreads)
fit_beta_kernel(const uint32_t *__restrict__ pa, const float *__restrict__ W, const float *__restrict__ alpha,
                const double *__restrict__ Gp, const double *__restrict__ Gq, int64_t d_in, int r,
                float *__restrict__ beta)
{
    extern __shared__ double sh[];
    const int n = (r + 1) & ~1;
    double *A = sh, *E = A + n * n, *cs = E + n * n, *h = cs + 2 * 64, *red = h + 64, *coef = red + (kFitThreads / 32) * 64;
    __shared__ double off_norm, all_norm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // h: rows strided over the threads, fixed-order tree
    double acc[64];
#pragma unroll
    for (int k = 0; k < 64; ++k) acc[k] = 0.0;
    for (int64_t i = tid; i < d_in; i += kFitThreads) {
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
    for (int e = tid; e < n * n; e += kFitThreads) {
        const int p = e / n, q = e - p * n;
        A[e] = (p < r && q < r) ? Gp[p * r + q] * Gq[p * r + q] : 0.0;     // Eq. beta-Schur
        E[e] = (p == q) ? 1.0 : 0.0;
    }
    __syncthreads();
    if (tid < 64) {
        double v = 0.0;
        for (int w = 0; w < kFitThreads / 32; ++w) v += red[w * 64 + tid];
        h[tid] = (tid < r) ? v : 0.0;
    }
    __syncthreads();

    // cyclic Jacobi, n / 2 disjoint rotations per round (round-robin pairing), at most 40 sweeps
    for (int sweep = 0; sweep < 40; ++sweep) {
        if (tid == 0) {
            double off = 0.0, all = 0.0;
            for (int p = 0; p < n; ++p)
                for (int q = 0; q < n; ++q) {
                    const double v = A[p * n + q] * A[p * n + q];
                    all += v;
                    if (p != q) off += v;
                }
            off_norm = off;
            all_norm = all;
        }
        __syncthreads();
        if (off_norm <= 1e-30 * all_norm) break;
        for (int round = 0; round < n - 1; ++round) {
            // pair m of this round: (n-1, round) for m = 0, else ((round+m) % (n-1), (round-m) mod (n-1))
            if (tid < n / 2) {
                const int m = tid;
                int p = (m == 0) ? n - 1 : (round + m) % (n - 1);
                int q = (m == 0) ? round : (round - m + (n - 1)) % (n - 1);
                const double apq = A[p * n + q];
                double c = 1.0, s = 0.0;
                if (apq != 0.0) {
                    const double theta = (A[q * n + q] - A[p * n + p]) / (2.0 * apq);
                    const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                    c = 1.0 / sqrt(t * t + 1.0);
                    s = t * c;
                }
                cs[2 * m] = c;
                cs[2 * m + 1] = s;
            }
            __syncthreads();
            // columns: A <- A J, E <- E J (task = row t, pair m)
            for (int task = tid; task < n * (n / 2); task += kFitThreads) {
                const int t = task / (n / 2), m = task - t * (n / 2);
                const int p = (m == 0) ? n - 1 : (round + m) % (n - 1);
                const int q = (m == 0) ? round : (round - m + (n - 1)) % (n - 1);
                const double c = cs[2 * m], s = cs[2 * m + 1];
                const double ap = A[t * n + p], aq = A[t * n + q];
                A[t * n + p] = c * ap - s * aq;
                A[t * n + q] = s * ap + c * aq;
                const double ep = E[t * n + p], eq = E[t * n + q];
                E[t * n + p] = c * ep - s * eq;
                E[t * n + q] = s * ep + c * eq;
            }
            __syncthreads();
            // rows: A <- J^T A (task = column t, pair m)
            for (int task = tid; task < n * (n / 2); task += kFitThreads) {
                const int t = task / (n / 2), m = task - t * (n / 2);
                const int p = (m == 0) ? n - 1 : (round + m) % (n - 1);
                const int q = (m == 0) ? round : (round - m + (n - 1)) % (n - 1);
                const double c = cs[2 * m], s = cs[2 * m + 1];
                const double ap = A[p * n + t], aq = A[q * n + t];
                A[p * n + t] = c * ap - s * aq;
                A[q * n + t] = s * ap + c * aq;
            }
            __syncthreads();
        }
    }
    __syncthreads();
    // beta = sum over eigenpairs with lambda > r eps lambda_max of (v^T h / lambda) v
    if (tid == 0) {
        double lmax = 0.0;
        for (int k = 0; k < n; ++k) lmax = fmax(lmax, A[k * n + k]);
        off_norm = (double)r * 2.220446049250313e-16 * lmax;
    }
    __syncthreads();
    if (tid < n) {
        const double lam = A[tid * n + tid];
        double dot = 0.0;
        for (int p = 0; p < r; ++p) dot += E[p * n + tid] * h[p];
        coef[tid] = (lam > off_norm) ? dot / lam : 0.0;
    }
    __syncthreads();
    if (tid < r) {
        double v = 0.0;
        for (int k = 0; k < n; ++k) v += E[tid * n + k] * coef[k];
        beta[tid] = (float)v;
    }
}

int padded_rank(int r) { return r <= 8 ? 8 : r <= 16 ? 16 : r <= 32 ? 32 : 64; }

struct FitWorkspace {
    float *W;          // d_in x r
    float *Vpart;      // chunks x r x d_out
    double *Gq, *Gp;   // r x r each
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
    w.Gq = reinterpret_cast<double *>(p + off); off += up((size_t)r * r * 8);
    w.Gp = reinterpret_cast<double *>(p + off); off += up((size_t)r * r * 8);
    w.bytes = off;
    return w;
}

size_t beta_smem(int r)
{
    const int n = (r + 1) & ~1;
    return sizeof(double) * (size_t)(2 * n * n + 2 * 64 + 64 + (kFitThreads / 32) * 64 + 64);
}

template <int RP>
void launch_row(const float *T, int64_t ld, const uint32_t *pb, const float *gamma, int64_t d_in, int64_t d_out, int r,
                float *W, cudaStream_t s)
{
    const int rows_per_block = kFitThreads / 32;
    fit_row_pass_kernel<RP><<<(unsigned)((d_in + rows_per_block - 1) / rows_per_block), kFitThreads, 0, s>>>(
        T, ld, pb, gamma, d_in, d_out, r, W);
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
                case 8:  launch_row<8>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
                case 16: launch_row<16>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
                case 32: launch_row<32>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
                default: launch_row<64>(target, ld, pb, s_out, d_in, d_out, r, w.W, stream); break;
            }
            fit_gram_kernel<1><<<r, kFitThreads, 0, stream>>>(pb, s_out, d_out, r, b_words, w.Gq);
            count_launch(2);
        }
        if (axes & LORDBA_FIT_ALPHA) {
            fit_alpha_kernel<<<(unsigned)((d_in + kFitThreads - 1) / kFitThreads), kFitThreads, 0, stream>>>(
                pa, w.W, w.Gq, s_r, d_in, r, s_in);
            count_launch();
        }
        if (axes & (LORDBA_FIT_BETA | LORDBA_FIT_GAMMA)) {
            fit_gram_kernel<0><<<r, kFitThreads, 0, stream>>>(pa, s_in, d_in, r, 0, w.Gp);
            count_launch();
        }
        if (axes & LORDBA_FIT_BETA) {
            fit_beta_kernel<<<1, kFitThreads, beta_smem(r), stream>>>(pa, w.W, s_in, w.Gp, w.Gq, d_in, r, s_r);
            count_launch();
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
