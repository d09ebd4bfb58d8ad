// Streaming tensor-core kernel of the LoRDBA adapter forward (bf16 activations),
// Eq. 8 / Eq. 9:
//
//   y[t,:] += s_out * ( B_sign ( s_r * ( A_sign ( s_in * x[t,:] ) ) ) )
//
// The branch moves 2 d_in + 4 d_out bytes per token and does 2 r (d_in + d_out)
// flops on them, so it is bound by HBM as long as the two sign products cost
// next to nothing and the memory system always has requests queued.
//
//   * One CTA owns `rows` <= 16 consecutive tokens (chosen on the host so that
//     the tiles of a call fill the SMs evenly) and needs no other CTA: the
//     16 x r intermediate lives in registers and shared memory.
//   * A producer warp streams the CTA's rows of x, then of y, through a ring of
//     shared-memory slots in chunks of `cw` columns with one bulk copy per row
//     (cp.async.bulk, completion on an mbarrier).  The chunk's slice of the
//     scale vector and of the packed carrier travels in the same slot, so there
//     are no other global loads.  The y chunks are requested while the first
//     product is still running: the memory system never drains between the two.
//   * Sixteen consumer warps each take one 64-column group of a chunk.  A lane
//     reads 16-byte pieces of two token rows from the slot straight into the
//     registers that are the A fragments of mma.sync.m16n8k16 (the K order of a
//     product is free, so the fragment's column pattern is re-labelled to make
//     every lane's columns contiguous); the D fragments of the second product
//     are re-labelled the same way, so y is updated and written to global memory
//     with 16-byte accesses.
//   * The sign bits are expanded to bf16 operands in registers: a B fragment of
//     the first product is (s_in as a bf16 hi/lo pair) XOR (sign-flip mask from a
//     256-entry table), one LOP3 per register; a B fragment of the second
//     product is +-1.0 looked up from 4 sign bits.  s_in and z = s_r * u are
//     split into bf16 hi + lo parts, so both products carry ~16 mantissa bits
//     into the float32 accumulators.
//
// Warps split the d_in axis for the first product (fixed-order reduction
// through shared memory, hence deterministic) and the d_out axis for the
// second.  gridDim.z > 1 splits the y chunks over several CTAs that each repeat
// the first product: used when a call has too few tokens to fill the GPU.
//
// Every mbarrier wait is bounded: after ~1 s it records a code in the device
// status word, raises the CTA's abort flag (all later waits return at once) and
// the kernel runs to its end.
#include <cuda_bf16.h>

#include <cstring>
#include <mutex>

#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kConsumerWarps = 16;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;      // + the producer warp
constexpr int kTile = 16;            // token rows of one MMA tile
constexpr int kGroup = 64;           // columns one warp handles per chunk (128 bytes per row)
constexpr int kMaxChunk = kGroup * kConsumerWarps;   // 1024 columns
constexpr int kRowPad = 64;          // bytes: consecutive rows of a slot start 64 bytes apart mod 128
constexpr int kMaxBatch = 32;        // projections per launch
constexpr int kMaxSlots = 8;
constexpr int kSmemBudget = 227 * 1024;
constexpr long long kWaitLimitCycles = 1500000000LL;

struct MmaBatch {
    lordba_proj p[kMaxBatch];
};

struct MmaParams {
    int64_t T;
    int rows;          // token rows per CTA tile (<= 16)
    int cwy;           // columns per y chunk: a multiple of 64, <= 1024 (x chunks are 1024 wide)
    int slots;         // ring depth
    int *status;       // device status word
};

// ---- shared-memory plan, same on host and device --------------------------------------------
struct SmemPlan {
    int row_stride;    // bytes between token rows of a slot
    int off_scale;     // slot offset of the chunk's float32 scales
    int off_bits;      // slot offset of the chunk's sign bytes
    int slot_bytes;
    int off_lut1, off_lut2, off_red, off_zh, off_zl, off_bar, total;
};

__host__ __device__ inline SmemPlan make_plan(int rp, int r, int slots)
{
    constexpr int cw = kMaxChunk;
    SmemPlan s;
    s.row_stride = cw * 2 + kRowPad;
    s.off_scale = kTile * s.row_stride;
    s.off_bits = s.off_scale + cw * 4;
    s.slot_bytes = (s.off_bits + cw * r / 8 + 127) / 128 * 128;
    const int ks = (rp + 15) / 16;
    s.off_lut1 = slots * s.slot_bytes;
    s.off_lut2 = s.off_lut1 + 256 * 16;
    s.off_red = s.off_lut2 + 16 * 8;
    s.off_zh = s.off_red + kConsumerWarps * kTile * rp * 4;
    s.off_zl = s.off_zh + kTile * ks * 8 * 4;
    s.off_bar = s.off_zl + kTile * ks * 8 * 4;
    s.total = s.off_bar + (2 * kMaxSlots + 2) * 8;
    return s;
}

// ---- PTX helpers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\n"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                 "selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// global -> shared bulk copy; both addresses 16-byte aligned, size a multiple of 16
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}

struct WaitCtx {
    volatile int *abort_flag;   // shared memory
    int *status;                // global status word
};

// Bounded wait.  Returns false once the CTA has given up.
__device__ __forceinline__ bool mbar_wait(const WaitCtx &w, uint32_t bar, uint32_t parity, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    if (*w.abort_flag) return false;
    const long long start = clock64();
    uint32_t spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (*w.abort_flag) return false;
            if (clock64() - start > kWaitLimitCycles) {
                atomicCAS(w.status, 0, code);
                *w.abort_flag = 1;
                return false;
            }
        }
    }
}

__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}

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

// The r sign bits of row j_local of a chunk's slice of B_sign (r/8 bytes per row, r % 8 == 0).
template <int RP>
__device__ __forceinline__ uint64_t b_row_bits(const uint8_t *bits, int j_local, int r)
{
    if (RP == 8) return bits[j_local];
    if (RP == 16) return reinterpret_cast<const uint16_t *>(bits)[j_local];
    if (r == 32) return reinterpret_cast<const uint32_t *>(bits)[j_local];
    if (r == 64) {
        const uint2 v = reinterpret_cast<const uint2 *>(bits)[j_local];
        return (uint64_t)v.x | ((uint64_t)v.y << 32);
    }
    const int nb = r >> 3;                       // 3, 5, 6 or 7 bytes
    uint64_t v = 0;
    for (int i = 0; i < nb; ++i) v |= (uint64_t)bits[j_local * nb + i] << (8 * i);
    return v;
}

// RP: rank padded to 8, 16, 32 or 64.
template <int RP>
__global__ void __launch_bounds__(kThreads, 1)
mma_forward_kernel(const __grid_constant__ MmaBatch batch, const __grid_constant__ MmaParams prm)
{
    constexpr int R8 = RP / 8;                 // 8-row blocks of A_sign = n-blocks of the first product
    constexpr int KS = (RP + 15) / 16;         // k-steps of the second product per z part
    constexpr int ZP = KS * 8;                 // bf16 pairs per token row of z
    constexpr bool kSplitAcc = (R8 <= 2);      // separate hi / lo accumulators: shorter MMA chains

    extern __shared__ __align__(128) uint8_t smem[];
    const lordba_proj &P = batch.p[blockIdx.y];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows = prm.rows, cwy = prm.cwy, S = prm.slots;
    constexpr int cwx = kMaxChunk;
    const int64_t t0 = (int64_t)blockIdx.x * rows;
    if (t0 >= prm.T) return;
    const int nt = (int)((prm.T - t0 < rows) ? (prm.T - t0) : rows);
    const int r = P.r;
    const int d_in = (int)P.d_in, d_out = (int)P.d_out;
    const SmemPlan plan = make_plan(RP, r, S);
    const uint32_t sm_base = smem_u32(smem);

    // chunk items: all x chunks, then this CTA's share of the y chunks
    const int n_x = (d_in + cwx - 1) / cwx;
    const int n_yc = (d_out + cwy - 1) / cwy;
    const int yc_begin = (int)((int64_t)blockIdx.z * n_yc / gridDim.z);
    const int yc_end = (int)((int64_t)(blockIdx.z + 1) * n_yc / gridDim.z);
    const int n_items = n_x + (yc_end - yc_begin);

    const uint32_t bar0 = sm_base + plan.off_bar;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kMaxSlots + s); };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + plan.off_bar + 2 * kMaxSlots * 8);
    const WaitCtx wctx{abort_flag, prm.status};

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), kConsumerWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    uint4 *lut1 = reinterpret_cast<uint4 *>(smem + plan.off_lut1);
    uint2 *lut2 = reinterpret_cast<uint2 *>(smem + plan.off_lut2);
    if (tid < 256) {
        // 8 sign bits (bit 1 = +1) -> XOR masks over four bf16 pairs (bit 0 => flip the sign)
        uint32_t m[4];
#pragma unroll
        for (int p = 0; p < 4; ++p)
            m[p] = (((tid >> (2 * p)) & 1) ? 0u : 0x8000u) | (((tid >> (2 * p + 1)) & 1) ? 0u : 0x80000000u);
        lut1[tid] = make_uint4(m[0], m[1], m[2], m[3]);
    } else if (tid < 256 + 16) {
        // 4 sign bits -> two registers of +-1.0 bf16 pairs
        const int t = tid - 256;
        const uint32_t b0 = 0x3f803f80u ^ ((t & 1) ? 0u : 0x8000u) ^ ((t & 2) ? 0u : 0x80000000u);
        const uint32_t b1 = 0x3f803f80u ^ ((t & 4) ? 0u : 0x8000u) ^ ((t & 8) ? 0u : 0x80000000u);
        lut2[t] = make_uint2(b0, b1);
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ================= producer warp: lanes 0..15 copy one token row each ===================
        const __nv_bfloat16 *xrow = static_cast<const __nv_bfloat16 *>(P.x) + (t0 + lane) * P.ldx;
        const __nv_bfloat16 *yrow = static_cast<const __nv_bfloat16 *>(P.y) + (t0 + lane) * P.ldy;
        const uint8_t *pa = reinterpret_cast<const uint8_t *>(P.packed_A);
        const uint8_t *pb = reinterpret_cast<const uint8_t *>(P.packed_B);
        for (int it = 0; it < n_items; ++it) {
            const int s = it % S;
            if (it >= S) mbar_wait(wctx, bar_empty(s), ((it / S) - 1) & 1u, kDevTmaWaitTimeout);
            if (*abort_flag) break;
            const bool is_x = it < n_x;
            const int cw = is_x ? cwx : cwy;
            const int col0 = is_x ? it * cwx : (yc_begin + (it - n_x)) * cwy;
            const int d = is_x ? d_in : d_out;
            const int cwv = (d - col0 < cw) ? (d - col0) : cw;              // valid columns, % 8 == 0
            const uint32_t bits_bytes = is_x ? (uint32_t)((cwv + kGroup - 1) / kGroup) * r * 8u
                                             : (uint32_t)cwv * r / 8u;
            const uint32_t slot = sm_base + s * plan.slot_bytes;
            if (lane == 0)
                mbar_arrive_expect_tx(bar_full(s), (uint32_t)nt * cwv * 2u + (uint32_t)cwv * 4u + bits_bytes);
            __syncwarp();
            if (lane < nt) {
                bulk_load(slot + lane * plan.row_stride, (is_x ? xrow : yrow) + col0, (uint32_t)cwv * 2u, bar_full(s));
            } else if (lane == 16) {
                bulk_load(slot + plan.off_scale, (is_x ? P.s_in : P.s_out) + col0, (uint32_t)cwv * 4u, bar_full(s));
            } else if (lane == 17) {
                const uint8_t *src = is_x ? pa + (size_t)(col0 / kGroup) * r * 8 : pb + (size_t)col0 * r / 8;
                bulk_load(slot + plan.off_bits, src, bits_bytes, bar_full(s));
            }
        }
    } else {
        // ================= consumer warps ========================================================
        const int g = lane >> 2, q = lane & 3;
        const bool v0 = g < nt, v1 = g + 8 < nt;    // this lane's two token rows exist
        const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
        const int gcol = warp * kGroup;             // first column of this warp's group within a chunk

        // ---- first product: u[t,k] = sum_i A_sign[k,i] s_in[i] x[t,i] -----------------------
        float acc[kSplitAcc ? 2 : 1][R8][4];
#pragma unroll
        for (int h = 0; h < (kSplitAcc ? 2 : 1); ++h)
#pragma unroll
            for (int a = 0; a < R8; ++a)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[h][a][e] = 0.0f;

        int it = 0;
        for (; it < n_x; ++it) {
            const int s = it % S;
            const bool ok = __all_sync(0xffffffffu, mbar_wait(wctx, bar_full(s), (it / S) & 1u, kDevMmaWaitTimeout));
            const int cwv = (d_in - it * cwx < cwx) ? (d_in - it * cwx) : cwx;
            if (gcol < cwv && ok) {
                const uint8_t *slot = smem + s * plan.slot_bytes;
                // this lane's columns: gcol + 8q .. +7 (half A) and gcol + 32 + 8q .. +7 (half B)
                const int ca = gcol + 8 * q, cb = ca + 32;
                const uint8_t *r0 = slot + g * plan.row_stride, *r1 = r0 + 8 * plan.row_stride;
                uint4 v[4];
                v[0] = (v0 && ca < cwv) ? *reinterpret_cast<const uint4 *>(r0 + 2 * ca) : zero4;
                v[1] = (v0 && cb < cwv) ? *reinterpret_cast<const uint4 *>(r0 + 2 * cb) : zero4;
                v[2] = (v1 && ca < cwv) ? *reinterpret_cast<const uint4 *>(r1 + 2 * ca) : zero4;
                v[3] = (v1 && cb < cwv) ? *reinterpret_cast<const uint4 *>(r1 + 2 * cb) : zero4;
                // s_in of the group as bf16 pairs (hi, lo): lane l converts columns 2l, 2l+1,
                // then every lane collects the pairs of its 16 columns
                uint32_t ph = 0u, pl = 0u;
                if (gcol + 2 * lane < cwv) {
                    const float2 sc = *reinterpret_cast<const float2 *>(slot + plan.off_scale + 4 * (gcol + 2 * lane));
                    split2(sc.x, sc.y, ph, pl);
                }
                uint32_t hA[4], hB[4], lA[4], lB[4];
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    hA[p] = __shfl_sync(0xffffffffu, ph, 4 * q + p);
                    hB[p] = __shfl_sync(0xffffffffu, ph, 16 + 4 * q + p);
                    lA[p] = __shfl_sync(0xffffffffu, pl, 4 * q + p);
                    lB[p] = __shfl_sync(0xffffffffu, pl, 16 + 4 * q + p);
                }
                const uint2 *blk = reinterpret_cast<const uint2 *>(slot + plan.off_bits) + warp * r;
#pragma unroll
                for (int a = 0; a < R8; ++a) {
                    int k = 8 * a + g;
                    if (k > r - 1) k = r - 1;                       // padded rank rows: result unused
                    const uint2 sb = blk[k];                         // the row's 64 sign bits of this block
                    const uint4 mA = lut1[(sb.x >> (8 * q)) & 0xffu];
                    const uint4 mB = lut1[(sb.y >> (8 * q)) & 0xffu];
                    float(&ch)[4] = acc[0][a];
                    float(&cl)[4] = acc[kSplitAcc ? 1 : 0][a];
                    mma_bf16(ch, v[0].x, v[2].x, v[0].y, v[2].y, hA[0] ^ mA.x, hA[1] ^ mA.y);
                    mma_bf16(cl, v[0].x, v[2].x, v[0].y, v[2].y, lA[0] ^ mA.x, lA[1] ^ mA.y);
                    mma_bf16(ch, v[0].z, v[2].z, v[0].w, v[2].w, hA[2] ^ mA.z, hA[3] ^ mA.w);
                    mma_bf16(cl, v[0].z, v[2].z, v[0].w, v[2].w, lA[2] ^ mA.z, lA[3] ^ mA.w);
                    mma_bf16(ch, v[1].x, v[3].x, v[1].y, v[3].y, hB[0] ^ mB.x, hB[1] ^ mB.y);
                    mma_bf16(cl, v[1].x, v[3].x, v[1].y, v[3].y, lB[0] ^ mB.x, lB[1] ^ mB.y);
                    mma_bf16(ch, v[1].z, v[3].z, v[1].w, v[3].w, hB[2] ^ mB.z, hB[3] ^ mB.w);
                    mma_bf16(cl, v[1].z, v[3].z, v[1].w, v[3].w, lB[2] ^ mB.z, lB[3] ^ mB.w);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
        }

        // ---- reduce u over the warps in a fixed order, z = s_r * u, split into bf16 hi + lo ---
        float *red = reinterpret_cast<float *>(smem + plan.off_red);
        uint32_t *zH = reinterpret_cast<uint32_t *>(smem + plan.off_zh);
        uint32_t *zL = reinterpret_cast<uint32_t *>(smem + plan.off_zl);
#pragma unroll
        for (int a = 0; a < R8; ++a) {
            float c[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) c[e] = kSplitAcc ? acc[0][a][e] + acc[kSplitAcc ? 1 : 0][a][e] : acc[0][a][e];
            float *d0 = red + ((warp * kTile + g) * RP + 8 * a + 2 * q);
            *reinterpret_cast<float2 *>(d0) = make_float2(c[0], c[1]);
            *reinterpret_cast<float2 *>(d0 + 8 * RP) = make_float2(c[2], c[3]);
        }
        consumer_sync();
        for (int idx = tid; idx < kTile * ZP; idx += kConsumerThreads) {
            const int tok = idx / ZP, pr = idx - tok * ZP;
            float u0 = 0.0f, u1 = 0.0f;
            if (2 * pr < RP) {
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
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
        consumer_sync();

        // ---- second product: y[t,j] += s_out[j] sum_k B_sign[j,k] z[t,k] ---------------------
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
        __nv_bfloat16 *yrow0 = static_cast<__nv_bfloat16 *>(P.y) + (t0 + g) * P.ldy;
        __nv_bfloat16 *yrow1 = yrow0 + 8 * P.ldy;

        for (; it < n_items; ++it) {
            const int s = it % S;
            const bool ok = __all_sync(0xffffffffu, mbar_wait(wctx, bar_full(s), (it / S) & 1u, kDevEpilogueWaitTimeout));
            const int col0 = (yc_begin + (it - n_x)) * cwy;
            const int cwv = (d_out - col0 < cwy) ? (d_out - col0) : cwy;
            if (gcol < cwv && ok) {
                const uint8_t *slot = smem + s * plan.slot_bytes;
                const uint8_t *bits = slot + plan.off_bits;
                // Output column of n-block (h, nb), accumulator column n = 2q + e:
                //   gcol + 32h + 8q + 2nb + e, so that a lane owns 8 consecutive columns per half.
                // As the holder of B-fragment column n = g this lane expands the signs of
                //   j = gcol + 32h + 8(g>>1) + 2nb + (g&1).
                float c[8][4];
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int e = 0; e < 4; ++e) c[i][e] = 0.0f;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                    for (int nb = 0; nb < 4; ++nb) {
                        int j = gcol + 32 * h + 8 * (g >> 1) + 2 * nb + (g & 1);
                        if (j > cwv - 1) j = cwv - 1;                  // columns past the end: unused
                        const uint64_t rb = b_row_bits<RP>(bits, j, r);
#pragma unroll
                        for (int ks = 0; ks < KS; ++ks) {
                            const uint32_t nib = (uint32_t)(rb >> (16 * ks + 4 * q)) & 0xfu;
                            const uint2 b = lut2[nib];
                            mma_bf16(c[h * 4 + nb], zh[ks][0], zh[ks][1], zh[ks][2], zh[ks][3], b.x, b.y);
                            mma_bf16(c[h * 4 + nb], zl[ks][0], zl[ks][1], zl[ks][2], zl[ks][3], b.x, b.y);
                        }
                    }
                }
                const uint8_t *r0 = slot + g * plan.row_stride, *r1 = r0 + 8 * plan.row_stride;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int col = gcol + 32 * h + 8 * q;
                    if (col < cwv) {
                        const float4 s0 = *reinterpret_cast<const float4 *>(slot + plan.off_scale + 4 * col);
                        const float4 s1 = *reinterpret_cast<const float4 *>(slot + plan.off_scale + 4 * col + 16);
                        const float so[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
                        for (int half = 0; half < 2; ++half) {          // token rows g and g + 8
                            if (half == 0 ? v0 : v1) {
                                const uint4 yv = *reinterpret_cast<const uint4 *>((half == 0 ? r0 : r1) + 2 * col);
                                const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w};
                                uint32_t ow[4];
#pragma unroll
                                for (int nb = 0; nb < 4; ++nb) {
                                    const float o0 = fmaf(so[2 * nb], c[h * 4 + nb][2 * half], lo_f(yw[nb]));
                                    const float o1 = fmaf(so[2 * nb + 1], c[h * 4 + nb][2 * half + 1], hi_f(yw[nb]));
                                    ow[nb] = pack2(o0, o1);
                                }
                                __stcs(reinterpret_cast<uint4 *>((half == 0 ? yrow0 : yrow1) + col0 + col),
                                       make_uint4(ow[0], ow[1], ow[2], ow[3]));
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
        }
    }

    // ---- teardown: after an abort, give copies that may still be in flight time to land ---------
    __syncthreads();
    if (*abort_flag) {
        const long long start = clock64();
        while (clock64() - start < 2000000LL) __nanosleep(1000);
    }
}

int padded_rank(int r) { return r <= 8 ? 8 : r <= 16 ? 16 : r <= 32 ? 32 : 64; }

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

template <int RP>
cudaError_t launch_one(const MmaBatch &b, const MmaParams &prm, dim3 grid, size_t smem, cudaStream_t stream)
{
    static std::once_flag once;
    static cudaError_t attr_rc = cudaSuccess;
    std::call_once(once, []() {
        attr_rc = cudaFuncSetAttribute(mma_forward_kernel<RP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kSmemBudget);
    });
    if (attr_rc != cudaSuccess) return attr_rc;
    mma_forward_kernel<RP><<<grid, kThreads, smem, stream>>>(b, prm);
    return cudaGetLastError();
}

}  // namespace

bool mma_supported(const lordba_proj &p, int64_t T, int dtype)
{
    if (dtype != LORDBA_BF16 || T < 1) return false;
    if (p.r % 8 != 0 || p.r < 8 || p.r > kMaxRank) return false;
    if (p.d_in % 8 != 0 || p.d_out % 8 != 0 || p.ldx % 8 != 0 || p.ldy % 8 != 0) return false;
    if (p.d_in > (1 << 30) || p.d_out > (1 << 30)) return false;
    // every bulk copy needs 16-byte aligned addresses and a size that is a multiple of 16:
    // rows of x / y, chunk slices of the scales, of packed_A (r * 8 bytes per 64 columns) and of
    // packed_B (r / 8 bytes per column; the last chunk ends at d_out * r / 8 bytes)
    if (reinterpret_cast<uintptr_t>(p.x) % 16 || reinterpret_cast<uintptr_t>(p.y) % 16) return false;
    if (reinterpret_cast<uintptr_t>(p.s_in) % 16 || reinterpret_cast<uintptr_t>(p.s_out) % 16 ||
        reinterpret_cast<uintptr_t>(p.packed_A) % 16 || reinterpret_cast<uintptr_t>(p.packed_B) % 16)
        return false;
    if ((p.d_out * p.r / 8) % 16 != 0) return false;
    return true;
}

int launch_forward_mma(const lordba_proj *projs, int n, int64_t T, int dtype, cudaStream_t stream)
{
    if (n == 0 || T == 0) return LORDBA_OK;
    if (dtype != LORDBA_BF16) return LORDBA_EUNSUPPORTED;
    int *status = device_status_word();
    if (!status) return LORDBA_ECUDA;
    const int sms = sm_count();
    for (int rp = 8; rp <= kMaxRank; rp *= 2) {
        MmaBatch b;
        int m = 0, max_r = 0;
        int64_t min_dout = (int64_t)1 << 40;
        for (int i = 0; i <= n; ++i) {
            const bool take = (i < n) && padded_rank(projs[i].r) == rp;
            if (take) {
                b.p[m++] = projs[i];
                if (projs[i].r > max_r) max_r = projs[i].r;
                if (projs[i].d_out < min_dout) min_dout = projs[i].d_out;
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
                // Few tokens: split the y chunks over several CTAs per tile (each repeats the
                // first product), with narrower chunks so that there is something to split.
                int64_t want_splits = sms / (tiles * m);
                if (want_splits < 1) want_splits = 1;
                int cw = kMaxChunk;
                while (cw > 128 && (min_dout + cw - 1) / cw < want_splits) cw /= 2;
                int64_t splits = (min_dout + cw - 1) / cw;
                if (splits > want_splits) splits = want_splits;
                if (splits > 64) splits = 64;

                MmaParams prm;
                prm.T = T; prm.rows = (int)rows; prm.cwy = cw; prm.status = status;
                int slots = kMaxSlots;
                while (slots > 2 && make_plan(rp, max_r, slots).total > kSmemBudget) --slots;
                const SmemPlan plan = make_plan(rp, max_r, slots);
                if (plan.total > kSmemBudget) return LORDBA_ECUDA;
                prm.slots = slots;
                const dim3 grid((unsigned)tiles, (unsigned)m, (unsigned)splits);
                cudaError_t e;
                switch (rp) {
                    case 8:  e = launch_one<8>(b, prm, grid, plan.total, stream); break;
                    case 16: e = launch_one<16>(b, prm, grid, plan.total, stream); break;
                    case 32: e = launch_one<32>(b, prm, grid, plan.total, stream); break;
                    default: e = launch_one<64>(b, prm, grid, plan.total, stream); break;
                }
                if (e != cudaSuccess) return LORDBA_ECUDA;
                count_launch();
                m = 0; max_r = 0; min_dout = (int64_t)1 << 40;
            }
        }
    }
    return LORDBA_OK;
}

}  // namespace lordba
