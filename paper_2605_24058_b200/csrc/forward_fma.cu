// CUDA-core (float32 FMA) kernel of the LoRDBA adapter forward, Eq. 8 / Eq. 9:
//
//   y[t,:] += s_out * ( B_sign ( s_r * ( A_sign ( s_in * x[t,:] ) ) ) )
//
// One CTA owns TT consecutive tokens and makes one pass: it streams the x rows
// with 128-bit loads, applies s_in, accumulates the r signed sums per token in
// registers (sign bits are expanded to +-1.0f through a 256-entry shared-memory
// table, one byte = 8 columns at a time), reduces across lanes with a
// transposing shuffle butterfly and across warps through shared memory in a
// fixed order, applies s_r, then walks the output columns expanding through
// B_sign, applies s_out and adds into y.  The T x r intermediate never leaves
// the SM.  This kernel takes every shape, pitch and alignment; it is the only
// kernel for float32 activations (no reduced-precision step anywhere).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstring>

#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxBatch = 32;      // projections per launch (kernel-parameter space)
constexpr int kAccPerThread = 64;  // TT * RP
constexpr int kMaxEll = 8;         // envelopes per adapter

struct FmaBatch {
    lordba_proj p[kMaxBatch];
    int64_t tokens[kMaxBatch];    // token rows of each projection
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// 8 consecutive elements of a row -> float; zero beyond n.  `vec` says that
// 16-byte loads are legal for this tensor (base and pitch aligned).
__device__ __forceinline__ void load8(const float *row, int64_t c0, int64_t n, bool vec, float out[8])
{
    if (vec && c0 + 8 <= n) {
        const float4 a = __ldcs(reinterpret_cast<const float4 *>(row + c0));
        const float4 b = __ldcs(reinterpret_cast<const float4 *>(row + c0 + 4));
        out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
        out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = (c0 + e < n) ? row[c0 + e] : 0.0f;
    }
}

__device__ __forceinline__ void load8(const __nv_bfloat16 *row, int64_t c0, int64_t n, bool vec,
                                      float out[8])
{
    if (vec && c0 + 8 <= n) {
        const uint4 a = __ldcs(reinterpret_cast<const uint4 *>(row + c0));
        out[0] = bf16_lo(a.x); out[1] = bf16_hi(a.x); out[2] = bf16_lo(a.y); out[3] = bf16_hi(a.y);
        out[4] = bf16_lo(a.z); out[5] = bf16_hi(a.z); out[6] = bf16_lo(a.w); out[7] = bf16_hi(a.w);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = (c0 + e < n) ? __bfloat162float(row[c0 + e]) : 0.0f;
    }
}

__device__ __forceinline__ void load8(const __half *row, int64_t c0, int64_t n, bool vec, float out[8])
{
    if (vec && c0 + 8 <= n) {
        const uint4 a = __ldcs(reinterpret_cast<const uint4 *>(row + c0));
        const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[e]));
            out[2 * e] = f.x;
            out[2 * e + 1] = f.y;
        }
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = (c0 + e < n) ? __half2float(row[c0 + e]) : 0.0f;
    }
}

__device__ __forceinline__ void store8(float *row, int64_t c0, int64_t n, bool vec, const float v[8])
{
    if (vec && c0 + 8 <= n) {
        __stcs(reinterpret_cast<float4 *>(row + c0), make_float4(v[0], v[1], v[2], v[3]));
        __stcs(reinterpret_cast<float4 *>(row + c0 + 4), make_float4(v[4], v[5], v[6], v[7]));
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (c0 + e < n) row[c0 + e] = v[e];
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
    return *reinterpret_cast<const uint32_t *>(&h);
}

__device__ __forceinline__ void store8(__nv_bfloat16 *row, int64_t c0, int64_t n, bool vec,
                                       const float v[8])
{
    if (vec && c0 + 8 <= n) {
        uint4 o;
        o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
        o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
        __stcs(reinterpret_cast<uint4 *>(row + c0), o);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (c0 + e < n) row[c0 + e] = __float2bfloat16_rn(v[e]);
    }
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);              // .x = lo (low half), .y = hi
    return *reinterpret_cast<const uint32_t *>(&h);
}

__device__ __forceinline__ void store8(__half *row, int64_t c0, int64_t n, bool vec, const float v[8])
{
    if (vec && c0 + 8 <= n) {
        uint4 o;
        o.x = pack_f16x2(v[0], v[1]); o.y = pack_f16x2(v[2], v[3]);
        o.z = pack_f16x2(v[4], v[5]); o.w = pack_f16x2(v[6], v[7]);
        __stcs(reinterpret_cast<uint4 *>(row + c0), o);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (c0 + e < n) row[c0 + e] = __float2half_rn(v[e]);
    }
}

// The r sign bits of output channel j (row j of B_sign) as the low bits of a
// 64-bit word: bits j*r .. j*r + r - 1 of the dense role-1 stream.
__device__ __forceinline__ uint64_t b_row_bits(const uint32_t *__restrict__ pb, int64_t n_words,
                                               int64_t j, int r)
{
    const int64_t bit = j * r;
    const int64_t w = bit >> 5;
    const int sh = (int)(bit & 31);
    const uint64_t w0 = __ldg(pb + w);
    const uint64_t w1 = (w + 1 < n_words) ? __ldg(pb + w + 1) : 0u;
    uint64_t win = ((w1 << 32) | w0) >> sh;
    if (sh != 0 && w + 2 < n_words) win |= (uint64_t)__ldg(pb + w + 2) << (64 - sh);
    return win;   // bits at and above r are ignored by the caller (their z is 0)
}

template <typename T, int RP>
__global__ void __launch_bounds__(kThreads)
fma_forward_kernel(const __grid_constant__ FmaBatch batch)
{
    const int64_t T_tokens = batch.tokens[blockIdx.y];
    constexpr int TT = kAccPerThread / RP;          // tokens per CTA
    const lordba_proj &P = batch.p[blockIdx.y];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int64_t t0 = (int64_t)blockIdx.x * TT;
    if (t0 >= T_tokens) return;
    const int nt = (int)((T_tokens - t0 < TT) ? (T_tokens - t0) : TT);

    const int r = P.r;
    const int64_t d_in = P.d_in, d_out = P.d_out;
    const T *__restrict__ x = static_cast<const T *>(P.x);
    T *__restrict__ y = static_cast<T *>(P.y);
    constexpr int kVecElems = 16 / (int)sizeof(T);
    const bool x_vec = (reinterpret_cast<uintptr_t>(x) % 16 == 0) && (P.ldx % kVecElems == 0);
    const bool y_vec = (reinterpret_cast<uintptr_t>(y) % 16 == 0) && (P.ldy % kVecElems == 0);

    // envelopes (Eq. 4): ell scale triples sharing the two carriers; ell = 1 is the canonical adapter
    const int ell = ((P.flags >> 8) & 0xf) + 1;

    __shared__ float4 lut[512];                     // byte -> 8 x (+-1.0f)
    __shared__ float red[kWarps][kAccPerThread];
    __shared__ __align__(16) float zs[kMaxEll][kAccPerThread];

    {
        float s[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) s[e] = ((tid >> e) & 1) ? 1.0f : -1.0f;
        lut[2 * tid] = make_float4(s[0], s[1], s[2], s[3]);
        lut[2 * tid + 1] = make_float4(s[4], s[5], s[6], s[7]);
    }
    __syncthreads();

    const uint8_t *__restrict__ pa = reinterpret_cast<const uint8_t *>(P.packed_A);
    // block-major layout: 64-column block b, row k -> 8 bytes at (b * r + k) * 8

    // ---- stage 1, per envelope: u[t,k] = sum_i A_sign[k,i] * (s_in[i] * x[t,i]), z = s_r * u ----
    for (int env = 0; env < ell; ++env) {
        const float *__restrict__ s_in = P.s_in + (int64_t)env * d_in;
        const bool s_vec = (reinterpret_cast<uintptr_t>(s_in) % 16 == 0);
        float acc[kAccPerThread];
#pragma unroll
        for (int i = 0; i < kAccPerThread; ++i) acc[i] = 0.0f;

        for (int64_t c0 = (int64_t)tid * 8; c0 < d_in; c0 += (int64_t)kThreads * 8) {
            float si[8];
            if (s_vec && c0 + 8 <= d_in) {
                const float4 a = __ldg(reinterpret_cast<const float4 *>(s_in + c0));
                const float4 b = __ldg(reinterpret_cast<const float4 *>(s_in + c0 + 4));
                si[0] = a.x; si[1] = a.y; si[2] = a.z; si[3] = a.w;
                si[4] = b.x; si[5] = b.y; si[6] = b.z; si[7] = b.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) si[e] = (c0 + e < d_in) ? __ldg(s_in + c0 + e) : 0.0f;
            }
            float xs[TT][8];
#pragma unroll
            for (int t = 0; t < TT; ++t) {
                if (t < nt) {
                    load8(x + (t0 + t) * P.ldx, c0, d_in, x_vec, xs[t]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) xs[t][e] *= si[e];
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) xs[t][e] = 0.0f;
                }
            }
#pragma unroll
            for (int k = 0; k < RP; ++k) {
                if (k < r) {
                    const uint32_t b = __ldg(pa + ((c0 >> 6) * r + k) * 8 + ((c0 & 63) >> 3));
                    const float4 lo = lut[2 * b], hi = lut[2 * b + 1];
#pragma unroll
                    for (int t = 0; t < TT; ++t) {
                        float a = acc[t * RP + k];
                        a = fmaf(xs[t][0], lo.x, a); a = fmaf(xs[t][1], lo.y, a);
                        a = fmaf(xs[t][2], lo.z, a); a = fmaf(xs[t][3], lo.w, a);
                        a = fmaf(xs[t][4], hi.x, a); a = fmaf(xs[t][5], hi.y, a);
                        a = fmaf(xs[t][6], hi.z, a); a = fmaf(xs[t][7], hi.w, a);
                        acc[t * RP + k] = a;
                    }
                }
            }
        }

        // reduce across the 32 lanes: transposing butterfly, 64 -> 2 values per lane
#pragma unroll
        for (int step = 16, n = kAccPerThread; step >= 1; step >>= 1, n >>= 1) {
            const bool upper = (lane & step) != 0;
            const int half = n >> 1;
#pragma unroll
            for (int i = 0; i < half; ++i) {
                const float send = upper ? acc[i] : acc[i + half];
                const float keep = upper ? acc[i + half] : acc[i];
                acc[i] = keep + __shfl_xor_sync(0xffffffffu, send, step);
            }
        }
        // lane now holds elements 2*lane and 2*lane+1 of the (t,k) grid
        red[warp][2 * lane] = acc[0];
        red[warp][2 * lane + 1] = acc[1];
        __syncthreads();
        if (tid < kAccPerThread) {
            float u = 0.0f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) u += red[w][tid];     // fixed order: deterministic
            const int k = tid % RP;
            zs[env][tid] = (k < r) ? u * __ldg(P.s_r + env * r + k) : 0.0f;       // z = s_r * u
        }
        __syncthreads();
    }

    // ---- stage 2: y[t,j] += sum_env s_out[env,j] * sum_k B_sign[j,k] * z[env,t,k] --------------
    const uint32_t *__restrict__ pb = P.packed_B;
    const int64_t b_words = (d_out * r + 31) / 32;

    for (int64_t j0 = (int64_t)tid * 8; j0 < d_out; j0 += (int64_t)kThreads * 8) {
        float yo[TT][8];
#pragma unroll
        for (int t = 0; t < TT; ++t) {
            if (t < nt) {
                load8(y + (t0 + t) * P.ldy, j0, d_out, y_vec, yo[t]);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) yo[t][e] = 0.0f;
            }
        }
        for (int env = 0; env < ell; ++env) {
            float z[kAccPerThread];
#pragma unroll
            for (int i = 0; i < kAccPerThread; i += 4) {
                const float4 q = *reinterpret_cast<const float4 *>(&zs[env][i]);
                z[i] = q.x; z[i + 1] = q.y; z[i + 2] = q.z; z[i + 3] = q.w;
            }
            const float *__restrict__ s_out = P.s_out + (int64_t)env * d_out;
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                const int64_t j = j0 + jj;
                if (j < d_out) {
                    float v[TT];
#pragma unroll
                    for (int t = 0; t < TT; ++t) v[t] = 0.0f;
                    const uint64_t bits = b_row_bits(pb, b_words, j, r);
#pragma unroll
                    for (int kc = 0; kc < RP / 8; ++kc) {
                        const uint32_t b = (uint32_t)(bits >> (8 * kc)) & 0xffu;
                        const float4 lo = lut[2 * b], hi = lut[2 * b + 1];
#pragma unroll
                        for (int t = 0; t < TT; ++t) {
                            const float *zt = &z[t * RP + kc * 8];
                            float a = v[t];
                            a = fmaf(zt[0], lo.x, a); a = fmaf(zt[1], lo.y, a);
                            a = fmaf(zt[2], lo.z, a); a = fmaf(zt[3], lo.w, a);
                            a = fmaf(zt[4], hi.x, a); a = fmaf(zt[5], hi.y, a);
                            a = fmaf(zt[6], hi.z, a); a = fmaf(zt[7], hi.w, a);
                            v[t] = a;
                        }
                    }
                    const float so = __ldg(s_out + j);
#pragma unroll
                    for (int t = 0; t < TT; ++t) yo[t][jj] = fmaf(so, v[t], yo[t][jj]);
                }
            }
        }
#pragma unroll
        for (int t = 0; t < TT; ++t)
            if (t < nt) store8(y + (t0 + t) * P.ldy, j0, d_out, y_vec, yo[t]);
    }
}

template <typename T>
const void *kernel_for(int rp)
{
    switch (rp) {
        case 8:  return reinterpret_cast<const void *>(&fma_forward_kernel<T, 8>);
        case 16: return reinterpret_cast<const void *>(&fma_forward_kernel<T, 16>);
        case 32: return reinterpret_cast<const void *>(&fma_forward_kernel<T, 32>);
        default: return reinterpret_cast<const void *>(&fma_forward_kernel<T, 64>);
    }
}

int emit_rank(const FmaBatch &b, int n, int rp, int dtype, LaunchSink &sink)
{
    const int tt = kAccPerThread / rp;
    int64_t T_tokens = 0;                          // the longest projection sets grid.x
    for (int i = 0; i < n; ++i) if (b.tokens[i] > T_tokens) T_tokens = b.tokens[i];
    const int64_t tiles = (T_tokens + tt - 1) / tt;
    LaunchRec rec;
    std::memset(&rec, 0, sizeof(rec));
    rec.func = (dtype == LORDBA_F32)    ? kernel_for<float>(rp)
               : (dtype == LORDBA_F16) ? kernel_for<__half>(rp)
                                       : kernel_for<__nv_bfloat16>(rp);
    rec.grid[0] = (unsigned)tiles; rec.grid[1] = (unsigned)n; rec.grid[2] = 1;
    rec.block = kThreads;
    rec.n_args = 1;
    rec.arg_bytes[0] = sizeof(FmaBatch);
    return sink.emit(rec, &b, nullptr);
}

int padded_rank(int r) { return r <= 8 ? 8 : r <= 16 ? 16 : r <= 32 ? 32 : 64; }

}  // namespace

int launch_forward_fma(const lordba_proj *projs, const int64_t *tokens, int64_t T, int n, const FamilySelector &sel,
                       LaunchSink &sink)
{
    // Group projections of equal padded rank into launches of at most kMaxBatch.
    for (int rp = 8; rp <= kMaxRank; rp *= 2) {
        FmaBatch b;
        int m = 0;
        for (int i = 0; i <= n; ++i) {
            const int64_t rows = (i < n) ? rows_of(tokens, T, i) : 0;
            const bool take = (i < n) && rows > 0 && padded_rank(projs[i].r) == rp &&
                              sel.family(projs[i], rows) == LORDBA_VARIANT_FMA;
            if (take) { b.tokens[m] = rows; b.p[m++] = projs[i]; }
            if (m == kMaxBatch || (i == n && m > 0)) {
                const int rc = emit_rank(b, m, rp, sel.dtype, sink);
                if (rc != LORDBA_OK) return rc;
                m = 0;
            }
        }
    }
    return LORDBA_OK;
}

}  // namespace lordba
