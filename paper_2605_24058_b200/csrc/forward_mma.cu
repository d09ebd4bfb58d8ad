// Register-streaming tensor-core kernel of the LoRDBA adapter forward (bf16
// activations), Eq. 8 / Eq. 9:
//
//   y[t,:] += s_out * ( B_sign ( s_r * ( A_sign ( s_in * x[t,:] ) ) ) )
//
// The branch moves 2 d_in + 4 d_out bytes per token and does 2 r (d_in + d_out)
// flops on them, so it is bound by HBM as long as the two sign products cost
// next to nothing.  This kernel therefore does three things:
//
//   * One CTA owns `rows` <= 16 consecutive tokens (chosen on the host so that
//     the tiles of a call fill the SMs evenly) and needs no other CTA: the
//     16 x r intermediate lives in registers and shared memory.
//   * x and y never pass through shared memory.  Each lane loads 16-byte pieces
//     of two token rows straight into the registers that are the A fragments of
//     mma.sync.m16n8k16 (the K order of a product is free, so the fragment's
//     column pattern is re-labelled to make every lane's columns contiguous);
//     the D fragments of the second product are re-labelled the same way, so y
//     is read, updated and written with 16-byte accesses as well.  All loads of
//     a lane are issued several column groups ahead.
//   * The sign bits are expanded to bf16 operands in registers: a B fragment of
//     the first product is (s_in as a bf16 hi/lo pair) XOR (sign-flip mask from a
//     256-entry table), one LOP3 per register; a B fragment of the second
//     product is +-1.0 looked up from 4 sign bits.  s_in and z = s_r * u are
//     split into bf16 hi + lo parts, so both products carry ~16 mantissa bits
//     into the float32 accumulators.
//
// Warps split the d_in axis for the first product (fixed-order reduction
// through shared memory, hence deterministic) and the d_out axis for the
// second.  gridDim.z > 1 splits d_out over several CTAs that each repeat the
// first product: used when a call has too few tokens to fill the GPU.
#include <cuda_bf16.h>

#include <cstring>
#include <mutex>

#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kTile = 16;            // token rows of one MMA tile
constexpr int kGroup = 64;           // columns one warp handles per step (128 bytes per row)
constexpr int kMaxBatch = 32;        // projections per launch
constexpr int kSmemLimit = 200 * 1024;

struct MmaBatch {
    lordba_proj p[kMaxBatch];
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
                 "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ float lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// v -> bf16 pair (hi parts) and bf16 pair (what the hi parts miss)
__device__ __forceinline__ void split2(float v0, float v1, uint32_t &hi, uint32_t &lo)
{
    hi = pack2(v0, v1);
    lo = pack2(v0 - lo_f(hi), v1 - hi_f(hi));
}

__device__ __forceinline__ uint4 ld_stream(const __nv_bfloat16 *p)
{
    return __ldcs(reinterpret_cast<const uint4 *>(p));
}

// The r sign bits of output channel j (dense role-1 stream: bit j*r + k), r a multiple of 8.
template <int RP>
__device__ __forceinline__ uint64_t b_row_bits(const uint32_t *__restrict__ pb, int64_t n_words, int64_t j, int r)
{
    if (RP == 8) return __ldg(reinterpret_cast<const uint8_t *>(pb) + j);
    if (RP == 16) return __ldg(reinterpret_cast<const uint16_t *>(pb) + j);
    if (r == 32) return __ldg(pb + j);
    if (r == 64) return (uint64_t)__ldg(pb + 2 * j) | ((uint64_t)__ldg(pb + 2 * j + 1) << 32);
    // 24, 40, 48, 56: byte-aligned rows inside the word stream
    const int64_t bit = j * r;
    const int64_t w = bit >> 5;
    const int sh = (int)(bit & 31);
    const uint64_t w0 = __ldg(pb + w);
    const uint64_t w1 = (w + 1 < n_words) ? __ldg(pb + w + 1) : 0u;
    uint64_t win = ((w1 << 32) | w0) >> sh;
    if (sh != 0 && w + 2 < n_words) win |= (uint64_t)__ldg(pb + w + 2) << (64 - sh);
    return win;
}

// RP: rank padded to 8, 16, 32 or 64.  PX / PY: column groups of x / y in flight per warp.
template <int RP, int PX, int PY>
__global__ void __launch_bounds__(kThreads, 1)
mma_forward_kernel(const __grid_constant__ MmaBatch batch, int64_t T_tokens, int rows)
{
    constexpr int R8 = RP / 8;                 // 8-row blocks of A_sign = n-blocks of the first product
    constexpr int KS = (RP + 15) / 16;         // k-steps of the second product per z part
    constexpr int ZP = KS * 8;                 // bf16 pairs per token row of z
    constexpr bool kSplitAcc = (R8 <= 2);      // separate hi / lo accumulators: shorter MMA chains

    extern __shared__ __align__(16) uint8_t smem[];
    const lordba_proj &P = batch.p[blockIdx.y];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, q = lane & 3;
    const int64_t t0 = (int64_t)blockIdx.x * rows;
    if (t0 >= T_tokens) return;
    const int nt = (int)((T_tokens - t0 < rows) ? (T_tokens - t0) : rows);
    const int r = P.r;
    const int d_in = (int)P.d_in, d_out = (int)P.d_out;
    const int ng_in = (d_in + kGroup - 1) / kGroup;
    const int ng_out = (d_out + kGroup - 1) / kGroup;
    const bool v0 = g < nt, v1 = g + 8 < nt;    // this lane's two token rows exist

    // shared memory: s_in as bf16 pairs (hi, lo), the two sign tables, the cross-warp buffers
    uint32_t *hiP = reinterpret_cast<uint32_t *>(smem);
    uint32_t *loP = hiP + ng_in * 32;
    uint4 *lut1 = reinterpret_cast<uint4 *>(loP + ng_in * 32);
    uint2 *lut2 = reinterpret_cast<uint2 *>(lut1 + 256);
    float *red = reinterpret_cast<float *>(lut2 + 16);
    uint32_t *zH = reinterpret_cast<uint32_t *>(red + kWarps * kTile * RP);
    uint32_t *zL = zH + kTile * ZP;

    // ---- first product: issue the first PX column groups of x before anything else ----------
    const __nv_bfloat16 *xrow0 = static_cast<const __nv_bfloat16 *>(P.x) + (t0 + g) * P.ldx;
    const __nv_bfloat16 *xrow1 = xrow0 + 8 * P.ldx;
    const int n_mine = (ng_in - warp + kWarps - 1) / kWarps;     // groups warp, warp + 16, ...
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
    auto load_x = [&](uint4 (&v)[4], int grp) {
        const int ca = grp * kGroup + 8 * q, cb = ca + 32;
        v[0] = (v0 && ca < d_in) ? ld_stream(xrow0 + ca) : zero4;
        v[1] = (v0 && cb < d_in) ? ld_stream(xrow0 + cb) : zero4;
        v[2] = (v1 && ca < d_in) ? ld_stream(xrow1 + ca) : zero4;
        v[3] = (v1 && cb < d_in) ? ld_stream(xrow1 + cb) : zero4;
    };
    uint4 xr[PX][4];
#pragma unroll
    for (int s = 0; s < PX; ++s) {
        if (s < n_mine) load_x(xr[s], warp + s * kWarps);
        else xr[s][0] = xr[s][1] = xr[s][2] = xr[s][3] = zero4;
    }

    // ---- tables ------------------------------------------------------------------------------
    for (int p = tid; p < ng_in * 32; p += kThreads) {
        const int c = 2 * p;
        float2 s = make_float2(0.0f, 0.0f);
        if (c < d_in) s = __ldg(reinterpret_cast<const float2 *>(P.s_in + c));
        uint32_t hi, lo;
        split2(s.x, s.y, hi, lo);
        hiP[p] = hi;
        loP[p] = lo;
    }
    if (tid < 256) {
        // 8 sign bits (bit 1 = +1) -> XOR masks over four bf16 pairs (bit 0 => flip the sign)
        uint32_t m[4];
#pragma unroll
        for (int p = 0; p < 4; ++p)
            m[p] = (((tid >> (2 * p)) & 1) ? 0u : 0x8000u) | (((tid >> (2 * p + 1)) & 1) ? 0u : 0x80000000u);
        lut1[tid] = make_uint4(m[0], m[1], m[2], m[3]);
    }
    if (tid < 16) {
        // 4 sign bits -> two registers of +-1.0 bf16 pairs
        const uint32_t b0 = 0x3f803f80u ^ ((tid & 1) ? 0u : 0x8000u) ^ ((tid & 2) ? 0u : 0x80000000u);
        const uint32_t b1 = 0x3f803f80u ^ ((tid & 4) ? 0u : 0x8000u) ^ ((tid & 8) ? 0u : 0x80000000u);
        lut2[tid] = make_uint2(b0, b1);
    }
    __syncthreads();

    // ---- first product: u[t,k] = sum_i A_sign[k,i] s_in[i] x[t,i] ---------------------------
    float acc[kSplitAcc ? 2 : 1][R8][4];
#pragma unroll
    for (int h = 0; h < (kSplitAcc ? 2 : 1); ++h)
#pragma unroll
        for (int a = 0; a < R8; ++a)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[h][a][e] = 0.0f;

    const uint2 *pa64 = reinterpret_cast<const uint2 *>(P.packed_A);
    const uint4 *hiP4 = reinterpret_cast<const uint4 *>(hiP);
    const uint4 *loP4 = reinterpret_cast<const uint4 *>(loP);

    auto consume_x = [&](const uint4 (&v)[4], int grp) {
        // this lane's columns: grp*64 + 8q .. +7 (half A) and grp*64 + 32 + 8q .. +7 (half B)
        const uint4 hA = hiP4[grp * 8 + q], hB = hiP4[grp * 8 + 4 + q];
        const uint4 lA = loP4[grp * 8 + q], lB = loP4[grp * 8 + 4 + q];
#pragma unroll
        for (int a = 0; a < R8; ++a) {
            int k = 8 * a + g;
            if (k > r - 1) k = r - 1;                            // padded rank rows: result unused
            const uint2 sb = __ldg(pa64 + ((size_t)grp * r + k));   // the row's 64 sign bits of this block
            const uint4 mA = lut1[(sb.x >> (8 * q)) & 0xffu];
            const uint4 mB = lut1[(sb.y >> (8 * q)) & 0xffu];
            float(&ch)[4] = acc[0][a];
            float(&cl)[4] = acc[kSplitAcc ? 1 : 0][a];
            mma_bf16(ch, v[0].x, v[2].x, v[0].y, v[2].y, hA.x ^ mA.x, hA.y ^ mA.y);
            mma_bf16(cl, v[0].x, v[2].x, v[0].y, v[2].y, lA.x ^ mA.x, lA.y ^ mA.y);
            mma_bf16(ch, v[0].z, v[2].z, v[0].w, v[2].w, hA.z ^ mA.z, hA.w ^ mA.w);
            mma_bf16(cl, v[0].z, v[2].z, v[0].w, v[2].w, lA.z ^ mA.z, lA.w ^ mA.w);
            mma_bf16(ch, v[1].x, v[3].x, v[1].y, v[3].y, hB.x ^ mB.x, hB.y ^ mB.y);
            mma_bf16(cl, v[1].x, v[3].x, v[1].y, v[3].y, lB.x ^ mB.x, lB.y ^ mB.y);
            mma_bf16(ch, v[1].z, v[3].z, v[1].w, v[3].w, hB.z ^ mB.z, hB.w ^ mB.w);
            mma_bf16(cl, v[1].z, v[3].z, v[1].w, v[3].w, lB.z ^ mB.z, lB.w ^ mB.w);
        }
    };

    for (int i0 = 0; i0 < n_mine; i0 += PX) {
#pragma unroll
        for (int s = 0; s < PX; ++s) {
            const int i = i0 + s;
            if (i < n_mine) {
                consume_x(xr[s], warp + i * kWarps);
                if (i + PX < n_mine) load_x(xr[s], warp + (i + PX) * kWarps);
            }
        }
    }

    // ---- second product, part 1: request the first y groups while u is being reduced ---------
    const int sp = blockIdx.z, n_sp = gridDim.z;
    const int og_begin = (int)((int64_t)sp * ng_out / n_sp);
    const int og_end = (int)((int64_t)(sp + 1) * ng_out / n_sp);
    const int m_mine = (og_end - og_begin - warp + kWarps - 1) / kWarps;
    __nv_bfloat16 *yrow0 = static_cast<__nv_bfloat16 *>(P.y) + (t0 + g) * P.ldy;
    __nv_bfloat16 *yrow1 = yrow0 + 8 * P.ldy;
    auto load_y = [&](uint4 (&v)[4], int grp) {
        const int ca = grp * kGroup + 8 * q, cb = ca + 32;
        v[0] = (v0 && ca < d_out) ? ld_stream(yrow0 + ca) : zero4;
        v[1] = (v0 && cb < d_out) ? ld_stream(yrow0 + cb) : zero4;
        v[2] = (v1 && ca < d_out) ? ld_stream(yrow1 + ca) : zero4;
        v[3] = (v1 && cb < d_out) ? ld_stream(yrow1 + cb) : zero4;
    };
    uint4 yr[PY][4];
#pragma unroll
    for (int s = 0; s < PY; ++s) {
        if (s < m_mine) load_y(yr[s], og_begin + warp + s * kWarps);
        else yr[s][0] = yr[s][1] = yr[s][2] = yr[s][3] = zero4;
    }

    // ---- reduce u over the warps in a fixed order, z = s_r * u, split into bf16 hi + lo ------
#pragma unroll
    for (int a = 0; a < R8; ++a) {
        float c[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) c[e] = kSplitAcc ? acc[0][a][e] + acc[kSplitAcc ? 1 : 0][a][e] : acc[0][a][e];
        float *d0 = red + ((warp * kTile + g) * RP + 8 * a + 2 * q);
        *reinterpret_cast<float2 *>(d0) = make_float2(c[0], c[1]);
        *reinterpret_cast<float2 *>(d0 + 8 * RP) = make_float2(c[2], c[3]);
    }
    __syncthreads();
    for (int idx = tid; idx < kTile * ZP; idx += kThreads) {
        const int tok = idx / ZP, pr = idx - tok * ZP;
        float u0 = 0.0f, u1 = 0.0f;
        if (2 * pr < RP) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float2 v = *reinterpret_cast<const float2 *>(red + ((w * kTile + tok) * RP + 2 * pr));
                u0 += v.x;
                u1 += v.y;
            }
        }
        const int k = 2 * pr;
        const float z0 = (k < r) ? u0 * __ldg(P.s_r + k) : 0.0f;
        const float z1 = (k + 1 < r) ? u1 * __ldg(P.s_r + k + 1) : 0.0f;
        uint32_t hi, lo;
        split2(z0, z1, hi, lo);
        zH[idx] = hi;
        zL[idx] = lo;
    }
    __syncthreads();

    // ---- second product: y[t,j] += s_out[j] sum_k B_sign[j,k] z[t,k] -------------------------
    // A fragments: k position (2q, 2q+1, 2q+8, 2q+9) of k-step s <-> ranks 16s + 4q + (0,1,2,3)
    uint32_t zh[KS][4], zl[KS][4];
#pragma unroll
    for (int s = 0; s < KS; ++s) {
        const uint2 h0 = *reinterpret_cast<const uint2 *>(zH + g * ZP + 8 * s + 2 * q);
        const uint2 h1 = *reinterpret_cast<const uint2 *>(zH + (g + 8) * ZP + 8 * s + 2 * q);
        const uint2 l0 = *reinterpret_cast<const uint2 *>(zL + g * ZP + 8 * s + 2 * q);
        const uint2 l1 = *reinterpret_cast<const uint2 *>(zL + (g + 8) * ZP + 8 * s + 2 * q);
        zh[s][0] = h0.x; zh[s][1] = h1.x; zh[s][2] = h0.y; zh[s][3] = h1.y;
        zl[s][0] = l0.x; zl[s][1] = l1.x; zl[s][2] = l0.y; zl[s][3] = l1.y;
    }
    const uint32_t *__restrict__ pb = P.packed_B;
    const int64_t b_words = ((int64_t)d_out * r + 31) / 32;

    auto consume_y = [&](const uint4 (&v)[4], int grp) {
        // Output column of n-block (h, nb), accumulator column n = 2q + e:
        //   grp*64 + 32h + 8q + 2nb + e, so that a lane owns 8 consecutive columns per half.
        // As the holder of B-fragment column n = g this lane expands the signs of
        //   j = grp*64 + 32h + 8(g>>1) + 2nb + (g&1).
        float c[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) c[i][e] = 0.0f;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
                int j = grp * kGroup + 32 * h + 8 * (g >> 1) + 2 * nb + (g & 1);
                if (j > d_out - 1) j = d_out - 1;                  // columns past the end: unused
                const uint64_t bits = b_row_bits<RP>(pb, b_words, j, r);
#pragma unroll
                for (int s = 0; s < KS; ++s) {
                    const uint32_t nib = (uint32_t)(bits >> (16 * s + 4 * q)) & 0xfu;
                    const uint2 b = lut2[nib];
                    mma_bf16(c[h * 4 + nb], zh[s][0], zh[s][1], zh[s][2], zh[s][3], b.x, b.y);
                    mma_bf16(c[h * 4 + nb], zl[s][0], zl[s][1], zl[s][2], zl[s][3], b.x, b.y);
                }
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int col = grp * kGroup + 32 * h + 8 * q;
            if (col < d_out) {
                const float4 s0 = __ldg(reinterpret_cast<const float4 *>(P.s_out + col));
                const float4 s1 = __ldg(reinterpret_cast<const float4 *>(P.s_out + col + 4));
                const float so[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
                for (int half = 0; half < 2; ++half) {              // token rows g and g + 8
                    if (half == 0 ? v0 : v1) {
                        const uint4 yv = v[2 * half + h];
                        const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w};
                        uint32_t ow[4];
#pragma unroll
                        for (int nb = 0; nb < 4; ++nb) {
                            const float o0 = fmaf(so[2 * nb], c[h * 4 + nb][2 * half], lo_f(yw[nb]));
                            const float o1 = fmaf(so[2 * nb + 1], c[h * 4 + nb][2 * half + 1], hi_f(yw[nb]));
                            ow[nb] = pack2(o0, o1);
                        }
                        __stcs(reinterpret_cast<uint4 *>((half == 0 ? yrow0 : yrow1) + col),
                               make_uint4(ow[0], ow[1], ow[2], ow[3]));
                    }
                }
            }
        }
    };

    for (int i0 = 0; i0 < m_mine; i0 += PY) {
#pragma unroll
        for (int s = 0; s < PY; ++s) {
            const int i = i0 + s;
            if (i < m_mine) {
                consume_y(yr[s], og_begin + warp + i * kWarps);
                if (i + PY < m_mine) load_y(yr[s], og_begin + warp + (i + PY) * kWarps);
            }
        }
    }
}

int padded_rank(int r) { return r <= 8 ? 8 : r <= 16 ? 16 : r <= 32 ? 32 : 64; }

size_t smem_bytes(int rp, int64_t d_in)
{
    const size_t ng = (size_t)((d_in + kGroup - 1) / kGroup);
    const size_t ks = (size_t)((rp + 15) / 16);
    return ng * 32 * 4 * 2 + 256 * 16 + 16 * 8 + (size_t)kWarps * kTile * rp * 4 + 2 * kTile * ks * 8 * 4;
}

int sm_count()
{
    static int n = []() {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1)
            v = 148;
        return v;
    }();
    return n;
}

template <int RP, int PX, int PY>
cudaError_t launch_one(const MmaBatch &b, dim3 grid, size_t smem, int64_t T, int rows, cudaStream_t stream)
{
    static std::once_flag once;
    static cudaError_t attr_rc = cudaSuccess;
    std::call_once(once, []() {
        attr_rc = cudaFuncSetAttribute(mma_forward_kernel<RP, PX, PY>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    });
    if (attr_rc != cudaSuccess) return attr_rc;
    mma_forward_kernel<RP, PX, PY><<<grid, kThreads, smem, stream>>>(b, T, rows);
    return cudaGetLastError();
}

}  // namespace

bool mma_supported(const lordba_proj &p, int64_t T, int dtype)
{
    if (dtype != LORDBA_BF16 || T < 1) return false;
    if (p.r % 8 != 0 || p.r < 8 || p.r > kMaxRank) return false;
    if (p.d_in % 8 != 0 || p.d_out % 8 != 0 || p.ldx % 8 != 0 || p.ldy % 8 != 0) return false;
    if (p.d_in > (1 << 30) || p.d_out > (1 << 30)) return false;
    if (reinterpret_cast<uintptr_t>(p.x) % 16 || reinterpret_cast<uintptr_t>(p.y) % 16) return false;
    if (reinterpret_cast<uintptr_t>(p.s_in) % 8 || reinterpret_cast<uintptr_t>(p.s_out) % 16 ||
        reinterpret_cast<uintptr_t>(p.packed_A) % 8)
        return false;
    return smem_bytes(padded_rank(p.r), p.d_in) <= (size_t)kSmemLimit;
}

int launch_forward_mma(const lordba_proj *projs, int n, int64_t T, int dtype, cudaStream_t stream)
{
    if (n == 0 || T == 0) return LORDBA_OK;
    if (dtype != LORDBA_BF16) return LORDBA_EUNSUPPORTED;
    const int sms = sm_count();
    for (int rp = 8; rp <= kMaxRank; rp *= 2) {
        MmaBatch b;
        int m = 0;
        int64_t max_din = 0, min_groups_out = 1 << 30;
        for (int i = 0; i <= n; ++i) {
            const bool take = (i < n) && padded_rank(projs[i].r) == rp;
            if (take) {
                b.p[m++] = projs[i];
                if (projs[i].d_in > max_din) max_din = projs[i].d_in;
                const int64_t go = (projs[i].d_out + kGroup - 1) / kGroup;
                if (go < min_groups_out) min_groups_out = go;
            }
            if (m == kMaxBatch || (i == n && m > 0)) {
                // Tile height: the smallest number of full waves of 16-row tiles, then the rows
                // per tile that spread the tokens evenly over those waves.
                const int64_t min_tiles = (int64_t)m * ((T + kTile - 1) / kTile);
                const int64_t waves = (min_tiles + sms - 1) / sms;
                int64_t tiles_target = waves * sms / m;
                if (tiles_target < 1) tiles_target = 1;
                int64_t rows = (T + tiles_target - 1) / tiles_target;
                if (rows > kTile) rows = kTile;
                if (rows < 1) rows = 1;
                const int64_t tiles = (T + rows - 1) / rows;
                // Few tokens: split d_out over several CTAs per tile (each repeats the first product).
                int64_t splits = sms / (tiles * m);
                if (splits > min_groups_out) splits = min_groups_out;
                if (splits > 64) splits = 64;
                if (splits < 1) splits = 1;
                const dim3 grid((unsigned)tiles, (unsigned)m, (unsigned)splits);
                const size_t smem = smem_bytes(rp, max_din);
                cudaError_t e;
                switch (rp) {
                    case 8:  e = launch_one<8, 4, 2>(b, grid, smem, T, (int)rows, stream); break;
                    case 16: e = launch_one<16, 4, 2>(b, grid, smem, T, (int)rows, stream); break;
                    case 32: e = launch_one<32, 3, 2>(b, grid, smem, T, (int)rows, stream); break;
                    default: e = launch_one<64, 2, 1>(b, grid, smem, T, (int)rows, stream); break;
                }
                if (e != cudaSuccess) return LORDBA_ECUDA;
                count_launch();
                m = 0; max_din = 0; min_groups_out = 1 << 30;
            }
        }
    }
    return LORDBA_OK;
}

}  // namespace lordba
