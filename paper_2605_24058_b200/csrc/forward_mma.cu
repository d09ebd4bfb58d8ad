// Streaming tensor-core kernel of the LoRDBA adapter forward (bf16 or float16
// activations), Eq. 8 / Eq. 9:
//
//   y[t,:] += s_out * ( B_sign ( s_r * ( A_sign ( s_in * x[t,:] ) ) ) )
//
// The branch moves 2 d_in + 4 d_out bytes per token and does 2 r (d_in + d_out)
// flops on them, so it is bound by HBM as long as the two sign products cost
// next to nothing and the memory system always has requests queued.
//
//   * One CTA owns `rows` <= 16 consecutive tokens (the host passes 16, the
//     height of an MMA tile: shorter tiles that fill the SMs more evenly were
//     measured slower) and needs no other CTA: the 16 x r intermediate lives
//     in registers and shared memory.
//   * A producer warp streams the CTA's rows of x, then of y, through a ring of
//     shared-memory slots, NW x 64 columns per item (NW = consumer warps), with
//     ONE tensor copy per item: the row-major matrix is described to TMA as a
//     3-D tensor (64 columns, rows, column groups), so a box of 64 x 16 x NW
//     lands as NW blocks of 2 KiB, [16 rows][128 bytes], 128-byte swizzled, one
//     block per consumer warp.  The item's slice of the scale vector and of the packed carrier
//     travels in the same slot (two small 2-D tensor copies), so there are no
//     other global loads.  The y items are requested while the first product is
//     still running: the memory system never drains between the two products.
//   * The NW consumer warps each take one 64-column group of an item.  NW = 16
//     with one CTA per SM for a lone call of a single wave of tiles; NW = 8 with
//     two CTAs per SM otherwise, so that one CTA's start-up and first-load
//     latency hide behind the other's streaming.  A lane
//     reads 16-byte pieces of two token rows from the slot straight into the
//     registers that are the A fragments of mma.sync.m16n8k16 (the K order of a
//     product is free, so the fragment's column pattern is re-labelled to make
//     every lane's 16 columns contiguous); the D fragments of the second product
//     are re-labelled the same way, so a lane updates 32 contiguous bytes of a y
//     row and writes them to global memory with one 256-bit store.
//   * The sign bits are expanded to bf16 operands in registers without tables:
//     a multiply by (2^a + 2^b) moves two sign bits to bits 15 and 31, and one
//     LOP3 folds them into the operand.  A B fragment of the first product is
//     s_in (as a bf16 hi/lo pair) with the signs XOR-ed in; a B fragment of the
//     second product is +-1.0.  s_in and z = s_r * u are split into bf16 hi + lo
//     parts, so both products carry ~16 mantissa bits into the float32
//     accumulators.  MMAs are issued k-step outermost, so that consecutive
//     ones go to different accumulators.
//   * float16 activations (the precision the method exports adapters in) use
//     the same kernel with half operands in the first product: s_in as a half
//     hi/lo pair, or, when the caller states that s_in holds half-precision
//     values (an adapter exported with fp16 scales), as one half, which halves
//     the tensor-core work of that product.  z stays a bf16 pair (its range is
//     not bounded by 65504) and the second product is unchanged.
//   * Multi-envelope adapters (Eq. 4: several scale triples over one pair of
//     carriers): the first product takes the envelopes EG at a time (as many as
//     keep EG x padded rank <= 64 partial sums per token row in registers), x
//     fragments and sign bits shared by the envelopes of a pass; an adapter with
//     more envelopes streams its x items once per group.  The second product
//     walks all envelopes with the same +-1 fragments and accumulates
//     sum_e s_out[e] * v_e on top of y in float32: one rounding.
//
// Warps split the d_in axis for the first product (fixed-order reduction
// through shared memory, hence deterministic) and the d_out axis for the
// second.  gridDim.z > 1 splits the y items over several CTAs: used when a call
// has too few tokens to fill the GPU.  Each of them repeats the first product,
// or, where d_in is long, they share it as clusters of 4 or 8 along grid z: a
// CTA streams only its part of d_in, stores its 16 x r partial sums into every
// cluster CTA's shared memory, arrives once on each one's barrier, and every
// CTA adds the parts in rank order once all have arrived (MmaParams::xsplit).
//
// A call that waits for its predecessor only because of y (the caller's promise
// LORDBA_PROJ_X_READY) requests its x items and runs the first product before
// it waits; the y items and everything that writes come after the wait.
//
// Every mbarrier wait is bounded: after ~1 s it records a code in the device
// status word, raises the CTA's abort flag (all later waits return at once) and
// the kernel runs to its end; a CTA whose first product is incomplete writes
// nothing, so every element of y is either its old value or the right new one.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstring>
#include <mutex>
#include <type_traits>

#include "lordba_internal.h"

namespace lordba {
namespace {

// Consumer warps per CTA (template parameter NW): 16 with one CTA per SM, or 8 with two CTAs per
// SM, so that one CTA's start-up and first-load latency hide behind the other's streaming.
// (Three CTAs per SM at 72 registers were measured slower: fewer slots per ring.)
constexpr int kTile = 16;            // token rows of one MMA tile = rows of a TMA box
constexpr int kGroup = 64;           // columns one warp handles per item (128 bytes per row)
constexpr int kBlockBytes = kTile * kGroup * 2;      // one warp's block of a slot: 2 KiB
constexpr int kMaxWarps = 16;
constexpr int kMaxBatch = 24;        // projections per launch (six tensor maps each)
constexpr int kMaxSlots = 8;
constexpr int kSmemBudget = 227 * 1024;
constexpr int kSmemBudgetHalf = 112 * 1024;      // two CTAs per SM

struct alignas(64) MmaProj {
    CUtensorMap x_map;     // bf16 (64, T, d_in / 64), box 64 x 16 x 16, 128-byte swizzle
    CUtensorMap y_map;     // bf16 (64, T, d_out / 64), box 64 x 16 x (cwy / 64), 128-byte swizzle
    CUtensorMap si_map;    // f32 (64, d_in / 64, ell), box 64 x NW x ell: the scales of an x item
    CUtensorMap so_map;    // f32 (64, d_out / 64, ell), box 64 x (cwy / 64) x ell
    CUtensorMap pa_map;    // u32 (16, d_in r / 512), box 16 x 2r: the sign bytes of an x item
    CUtensorMap pb_map;    // u32 (16, d_out r / 512), box 16 x (cwy r / 512)
    const float *s_r;
    uint16_t *y;           // 16-bit elements: bfloat16 or half
    int64_t ldy;
    int64_t T;             // token rows of this projection (projections of a launch may differ)
    int d_in, d_out, r;
    int y_vec32;           // y rows are 32-byte aligned: 256-bit stores
};

struct MmaBatch {
    MmaProj p[kMaxBatch];
};

struct MmaParams {
    int rows;          // token rows per CTA tile (<= 16)
    int cwy;           // columns per y item: a multiple of 64, <= 1024 (x items are 1024 wide)
    int slots;         // ring depth
    int wait_prev;     // 1: the previous kernel of the stream must be complete before any global access
    int skip_item;     // -1; the test-hooks build can name one item whose copy request is left out
    int xsplit;        // C > 1 (single-envelope launches of few tiles): the CTAs are launched as clusters of C
                       // along grid z; CTA c of a cluster takes every x item of its share of the d_in axis
                       // only, and the partial sums of u go round the cluster through distributed shared memory
    int x_ready;       // 1 (only with wait_prev): x and the adapter were final before the previous kernel began,
                       // so the x items are requested and the first product runs before the wait for it;
                       // y is touched only afterwards
    int spread_issue;  // 1: the first requests are issued by one lane each instead of one after the other
    int gate_y;        // g > 0: the y items that fit the ring at the start are requested only once x item
                       // g - 1 has landed, so that the x items, which the first product waits for, do not
                       // share the memory system with them from the start (0: everything is requested at once)
    int ell;           // envelopes of the adapters of this launch (Eq. 4); the first product takes them
                       // EG at a time, streaming the x items once per group
    int *status;       // device status word
};

// ---- shared-memory plan, same on host and device --------------------------------------------
struct SmemPlan {
    int off_scale;     // slot offset of the item's float32 scales
    int off_bits;      // slot offset of the item's sign bytes
    int slot_bytes;    // multiple of 1024 (swizzle atom)
    int off_red, off_zh, off_zl, off_ux, off_bar, total;
};

// nw: consumer warps = 64-column groups per item; cwy: columns of a y item
// eg: envelopes (scale triples) per pass of the first product: eg rows of scales per x item, eg
// partial sums; ell: all envelopes of the adapter: ell rows of scales per y item, ell z tiles
// xsplit: CTAs of a cluster that share the first product (1: none): one tile of partial u per CTA
__host__ __device__ inline SmemPlan make_plan(int nw, int rp, int r, int slots, int eg, int ell, int cwy, int xsplit = 1)
{
    SmemPlan s;
    s.off_scale = nw * kBlockBytes;
    const int sx = eg * nw * kGroup, sy = ell * cwy;
    s.off_bits = s.off_scale + (sx > sy ? sx : sy) * 4;
    s.slot_bytes = (s.off_bits + nw * kGroup * r / 8 + 1023) / 1024 * 1024;
    const int ks = (rp + 15) / 16;
    s.off_red = slots * s.slot_bytes;
    s.off_zh = s.off_red + eg * nw * kTile * rp * 4;
    s.off_zl = s.off_zh + ell * kTile * ks * 8 * 4;
    s.off_ux = s.off_zl + ell * kTile * ks * 8 * 4;
    s.off_bar = s.off_ux + (xsplit > 1 ? xsplit * kTile * ks * 16 * 4 : 0);
    s.total = s.off_bar + (2 * kMaxSlots + 2) * 8 + 1024;    // + slack to align the base to 1 KiB
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
// ---- cluster helpers (launches whose CTAs share the first product) ----
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t v; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(v)); return v;
}
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank)
{
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f2(uint32_t addr, float a, float b)
{
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
// arrive on a barrier of any CTA of the cluster (address from mapa).  Relaxed: the stores that the
// arrival publishes were fenced at cluster scope by the threads that made them, before the CTA
// barrier that precedes this arrival.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;" ::: "memory");
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
// Tiled tensor copies global -> shared (coordinates innermost first; c0 * element size % 16 == 0).
// Plain (untiled) bulk copies are not used: they were measured at ~8 bytes per cycle here,
// against more than 100 for a tiled box.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void st_global_256(void *p, const uint32_t (&a)[4], const uint32_t (&b)[4])
{
    asm volatile("st.global.L1::no_allocate.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(p), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]), "r"(b[2]), "r"(b[3])
                 : "memory");
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

// The same for a barrier on which other CTAs of the cluster arrive (acquire at cluster scope).
__device__ __forceinline__ bool mbar_wait_cluster(const WaitCtx &w, uint32_t bar, uint32_t parity, int code)
{
    const long long start = clock64();
    uint32_t spins = 0;
    for (;;) {
        uint32_t ok;
        asm volatile("{\n.reg .pred p;\n"
                     "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
                     "selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
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

template <int kThreadsInBarrier>
__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kThreadsInBarrier) : "memory");
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
                 "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 "
                 "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (d0, d1) += (a0, a1) * (b0, b1): one packed fp32 FMA, each half rounded like fmaf
__device__ __forceinline__ void fma2(float &d0, float &d1, float a0, float a1, float b0, float b1)
{
    asm("{\n.reg .b64 ra, rb, rc;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\nmov.b64 rc, {%0, %1};\n"
        "fma.rn.f32x2 rc, ra, rb, rc;\nmov.b64 {%0, %1}, rc;\n}"
        : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
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

// The same for IEEE halves.  The low parts go subnormal for |v| below about 2^-3 and then keep an
// absolute precision of 2^-25: still beyond what a half-precision output can show.
__device__ __forceinline__ uint32_t pack2h(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ float2 unpack2h(uint32_t w) { return __half22float2(*reinterpret_cast<const __half2 *>(&w)); }
__device__ __forceinline__ void split2h(float v0, float v1, uint32_t &hi, uint32_t &lo)
{
    hi = pack2h(v0, v1);
    const float2 h = unpack2h(hi);
    lo = pack2h(v0 - h.x, v1 - h.y);
}

// Sign bits (bit 1 = +1) -> sign-flip masks of bf16 (or half) pairs.  b holds sign bits in its low byte
// (nothing above bit 7); pair p takes bits 2p and 2p+1.  b * (2^(15-2p) + 2^(30-2p)) is two
// disjoint shifted copies of b that put bit 2p at position 15 and bit 2p+1 at position 31; the
// caller keeps only those two positions, inverted (a 0 bit flips the sign).
constexpr uint32_t kSignBits = 0x80008000u;
__device__ __forceinline__ uint32_t pair_bits(uint32_t b, int p)
{
    return b * ((1u << (15 - 2 * p)) + (1u << (30 - 2 * p)));
}
__device__ __forceinline__ uint32_t with_signs(uint32_t operand, uint32_t bits)
{
    return operand ^ (~bits & kSignBits);
}

// The r sign bits of row j_local of an item's slice of B_sign, which is the dense bit stream of
// the rows.  GEN = false: r is 8, 16, 32 or 64 and a row is one aligned load.  GEN = true (any
// other rank, its own instantiations so that the common ranks keep their code): a row starts at
// bit j_local * r and is cut out of the two or three aligned words that hold it (the stream
// starts word-aligned; a word past its end is still inside the slot).  Bits above the row's r
// belong to other rows and are harmless: those ranks of z are zero.
template <int RP, bool GEN>
__device__ __forceinline__ uint64_t b_row_bits(const uint8_t *bits, int j_local, int r)
{
    if (!GEN) {
        if (RP == 8) return bits[j_local];
        if (RP == 16) return reinterpret_cast<const uint16_t *>(bits)[j_local];
        if (RP == 32) return reinterpret_cast<const uint32_t *>(bits)[j_local];
        const uint2 v = reinterpret_cast<const uint2 *>(bits)[j_local];
        return (uint64_t)v.x | ((uint64_t)v.y << 32);
    }
    const int bit = j_local * r, sh = bit & 31;
    const uint32_t *w = reinterpret_cast<const uint32_t *>(bits) + (bit >> 5);
    uint64_t v = ((uint64_t)w[0] | ((uint64_t)w[1] << 32)) >> sh;
    if (RP > 32 && sh > 0) v |= (uint64_t)w[2] << (64 - sh);
    return v;
}

// Element type of x and y, and how s_in enters the first product.
enum IoKind {
    kIoBf16 = 0,      // bfloat16; s_in as a bf16 hi + lo pair (two passes over the tensor cores)
    kIoF16 = 1,       // IEEE half; s_in as a half hi + lo pair (two passes)
    kIoF16Exact = 2   // IEEE half; s_in stated to be exact in half precision: one pass
};

// RP: rank padded to 8, 16, 32 or 64.  EG: envelopes per pass of the first product (EG * RP <= 64:
// their partial sums live in registers); an adapter with more envelopes than that streams its x
// items once per group of EG, the y items once.
// EGT = 0 stands for "one envelope per pass, several envelopes in all" (rank above 32), EGT = 1 for
// the single-envelope adapter, whose code carries no envelope loops at all.
// EGT_ = -1 is the single-envelope kernel whose CTAs share the first product as clusters
// (MmaParams::xsplit), an instantiation of its own so that the others carry none of that code.
template <int RP, int NW, int EGT_, int IO, bool GEN>
__global__ void __launch_bounds__(NW * 32 + 32, NW == 16 ? 1 : 2)
mma_forward_kernel(const __grid_constant__ MmaBatch batch, const __grid_constant__ MmaParams prm)
{
    constexpr bool kClusters = (EGT_ == -1);
    constexpr int EGT = kClusters ? 1 : EGT_;
    constexpr int EG = (EGT == 0) ? 1 : EGT;
    constexpr bool kHalf = (IO != kIoBf16);     // x, y and the first product's operands are halves
    constexpr bool kLoPass = (IO != kIoF16Exact);
    constexpr int R8 = RP / 8;                 // 8-row blocks of A_sign = n-blocks of the first product
    constexpr int KS = (RP + 15) / 16;         // k-steps of the second product per z part
    constexpr int ZP = KS * 8;                 // bf16 pairs per token row of z
    constexpr bool kSplitAcc = (EG * R8 <= 2); // separate hi / lo accumulators: shorter MMA chains
    constexpr int kConsumerWarps = NW, kConsumerThreads = NW * 32;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // swizzle atoms: 1 KiB
    const MmaProj &P = batch.p[blockIdx.y];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows = prm.rows, cwy = prm.cwy, S = prm.slots;
    constexpr int cwx = NW * kGroup;
    const int64_t t0 = (int64_t)blockIdx.x * rows;
    if (t0 >= P.T) return;
    const int nt = (int)((P.T - t0 < rows) ? (P.T - t0) : rows);
    const int r = P.r;
    const int d_in = P.d_in, d_out = P.d_out;
    const int ell = (EGT == 1) ? 1 : prm.ell;
    const int n_groups = (EGT == 1) ? 1 : (ell + EG - 1) / EG;
    // CTAs of a cluster along grid z share the first product (single-envelope launches only)
    const int xsplit = kClusters ? prm.xsplit : 1;
    const SmemPlan plan = make_plan(NW, RP, r, S, EG, ell, cwy, xsplit);
    const uint32_t sm_base = smem_u32(smem);

    // items: the x chunks (once per envelope group; with a cluster this CTA's share of them, a
    // contiguous range), then this CTA's share of the y chunks
    const int n_x_all = (d_in + cwx - 1) / cwx;
    const int xrank = xsplit > 1 ? (int)cluster_ctarank() : 0;
    const int x_first = (int)((int64_t)xrank * n_x_all / xsplit);
    const int n_x = (int)((int64_t)(xrank + 1) * n_x_all / xsplit) - x_first;
    const int n_xi = n_groups * n_x;
    const int n_yc = (d_out + cwy - 1) / cwy;
    const int yc_begin = (int)((int64_t)blockIdx.z * n_yc / gridDim.z);
    const int yc_end = (int)((int64_t)(blockIdx.z + 1) * n_yc / gridDim.z);
    const int n_items = n_xi + (yc_end - yc_begin);

    const uint32_t bar0 = sm_base + plan.off_bar;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kMaxSlots + s); };
    const uint32_t bar_ux = bar0 + 8u * (2 * kMaxSlots + 1);    // partial sums of the whole cluster have arrived
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + plan.off_bar + 2 * kMaxSlots * 8);
    const WaitCtx wctx{abort_flag, prm.status};

    // Programmatic dependent launch.  A kernel that must see its predecessor (wait_prev) sets up,
    // waits for it, and only then lets its own successor in: whatever ran before it is complete
    // by the time anything after it starts.  A kernel that the caller declared independent of the
    // calls before it lets its successor in at once, streams without waiting, and waits for its
    // predecessor just before it exits, so that "this grid is complete" still implies "everything
    // before it is complete".
    if (!prm.wait_prev) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp == kConsumerWarps) {
        // the producer warp's first lane prepares the barriers; everybody else meets the warp at the
        // barrier below
        if (lane == 0) {
            for (int s = 0; s < S; ++s) {
                mbar_init(bar_full(s), 1);
                mbar_init(bar_empty(s), kConsumerWarps);
            }
            if (xsplit > 1) mbar_init(bar_ux, (uint32_t)xsplit);   // one arrival per CTA of the cluster
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        if (prm.wait_prev && !prm.x_ready) {
            // everything before this line overlapped the previous kernel; nothing after it may
            // (every lane that is going to request data waits itself)
            asm volatile("griddepcontrol.wait;" ::: "memory");
            if (lane == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        }
    }
    auto issue_item = [&](int it, int s) {       // one thread; s = it % S
        const bool is_x = it < n_xi;
        const int cw = is_x ? cwx : cwy;
        const int grp = is_x ? it / n_x : 0;       // the envelope group this pass over x belongs to
        const int col0 = is_x ? (x_first + it - grp * n_x) * cwx : (yc_begin + (it - n_xi)) * cwy;
        // a box is always whole: what lies past the tensor (columns, envelopes) is filled with zeros and counted
        const uint32_t bytes = (uint32_t)(cw / kGroup) * kBlockBytes + (uint32_t)(is_x ? EG : ell) * cw * 4u +
                               (uint32_t)cw * r / 8u;
        const uint32_t slot = sm_base + s * plan.slot_bytes;
        if (it == prm.skip_item) return;          // test-hooks build only: nothing is requested, nothing lands
        mbar_arrive_expect_tx(bar_full(s), bytes);
        tma_load_3d(slot, is_x ? &P.x_map : &P.y_map, 0, (int)t0, col0 / kGroup, bar_full(s));
        tma_load_3d(slot + plan.off_scale, is_x ? &P.si_map : &P.so_map, 0, col0 / kGroup, grp * EG, bar_full(s));
        tma_load_2d(slot + plan.off_bits, is_x ? &P.pa_map : &P.pb_map, 0, col0 * r / 512, bar_full(s));
    };
    const int n_first = n_items < S ? n_items : S;
    const int n_eager = ((prm.gate_y || prm.x_ready) && n_xi < n_first) ? n_xi : n_first;
    // The first requests (n_eager <= n_first <= S <= 32).  A tensor copy takes its issuing thread some
    // 50 ns and the ring's first fill is up to 18 of them: the cluster launches of few tiles, which
    // are all latency, have one lane of the producer warp issue each item (a decode-sized layer call
    // that waits for its predecessor: 5.9 -> 5.65 us); everywhere else the items go out in order from
    // one lane (the other way measured 2 - 7 % behind where the memory system is the limit).
    if (warp == kConsumerWarps) {
        if (prm.spread_issue) {
            if (lane < n_eager) issue_item(lane, lane);
        } else if (lane == 0) {
            for (int it = 0; it < n_eager; ++it) issue_item(it, it);
        }
    }
    __syncthreads();
    // every CTA of the cluster has initialised its barriers before any of them arrives on another's
    // (all CTAs of a cluster have the same tile and projection: none has left above)
    if (xsplit > 1) cluster_sync_all();

    if (warp == kConsumerWarps) {
        // ================= producer warp: one lane refills the slots as they are released ========
        if (lane == 0) {
            // item n_first is the first to reuse a slot: slot 0, first release phase
            int s = 0;
            uint32_t eph = 0;
            if (prm.x_ready) {
                // what was requested so far is x and the adapter; from here on y, which the
                // previous kernel may have written: wait for it, then let the successor in
                asm volatile("griddepcontrol.wait;" ::: "memory");
                asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            }
            if (n_eager < n_first &&
                (n_eager == 0 || prm.gate_y == 0 ||
                 mbar_wait(wctx, bar_full(prm.gate_y - 1 < n_eager ? prm.gate_y - 1 : n_eager - 1), 0u, kDevTmaWaitTimeout)))
                for (int it = n_eager; it < n_first; ++it) issue_item(it, it);
            for (int it = n_first; it < n_items; ++it) {
                if (!mbar_wait(wctx, bar_empty(s), eph, kDevTmaWaitTimeout)) break;
                issue_item(it, s);
                if (++s == S) { s = 0; eph ^= 1u; }
            }
        }
    } else {
        // ================= consumer warps ========================================================
        const int g = lane >> 2, q = lane & 3;
        const bool v0 = g < nt, v1 = g + 8 < nt;    // this lane's two token rows belong to the tile
        const int gcol = warp * kGroup;             // first column of this warp's group within an item
        // this lane's pieces of its two rows inside the warp's 2 KiB block (128-byte swizzle:
        // 16-byte piece c of row i sits at piece c ^ (i & 7))
        const int off_r0 = warp * kBlockBytes + g * 128, off_r1 = off_r0 + 8 * 128;
        const int pc0 = ((2 * q) ^ g) * 16, pc1 = ((2 * q + 1) ^ g) * 16;

        // ---- first product: u[t,k] = sum_i A_sign[k,i] s_in[i] x[t,i] -----------------------
        float *red = reinterpret_cast<float *>(smem + plan.off_red);
        uint32_t *zH = reinterpret_cast<uint32_t *>(smem + plan.off_zh);
        uint32_t *zL = reinterpret_cast<uint32_t *>(smem + plan.off_zl);
        int it = 0;
        int s = 0;                 // ring slot of item `it` and the phase of its barrier, carried
        uint32_t sph = 0;          // along instead of recomputed by division
        for (int grp = 0; grp < n_groups; ++grp) {
        float acc[EG][kSplitAcc ? 2 : 1][R8][4];
#pragma unroll
        for (int env = 0; env < EG; ++env)
#pragma unroll
            for (int h = 0; h < (kSplitAcc ? 2 : 1); ++h)
#pragma unroll
                for (int a = 0; a < R8; ++a)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[env][h][a][e] = 0.0f;

        for (int xc = 0; xc < n_x; ++xc, ++it) {
            const bool ok = __all_sync(0xffffffffu, mbar_wait(wctx, bar_full(s), sph, kDevMmaWaitTimeout));
            const int cwv = (d_in - (x_first + xc) * cwx < cwx) ? (d_in - (x_first + xc) * cwx) : cwx;
            if (gcol < cwv && ok) {
                const uint8_t *slot = smem + s * plan.slot_bytes;
                // this lane's columns: gcol + 16q .. +7 (piece A) and gcol + 16q + 8 .. +15 (piece B);
                // rows past the tile are other tokens or zero fill and only reach unused outputs
                const uint4 xa0 = *reinterpret_cast<const uint4 *>(slot + off_r0 + pc0);
                const uint4 xb0 = *reinterpret_cast<const uint4 *>(slot + off_r0 + pc1);
                const uint4 xa1 = *reinterpret_cast<const uint4 *>(slot + off_r1 + pc0);
                const uint4 xb1 = *reinterpret_cast<const uint4 *>(slot + off_r1 + pc1);
                // the warp's block of the carrier: r rows of 64 sign bits; this lane's 16 columns are
                // half-word q of a row
                const uint16_t *blk = reinterpret_cast<const uint16_t *>(slot + plan.off_bits) + warp * r * 4 + q;
                uint32_t bytes[R8];                                  // sign bits of this lane's 16 columns
#pragma unroll
                for (int a = 0; a < R8; ++a) {
                    int k = 8 * a + g;
                    if (k > r - 1) k = r - 1;                       // padded rank rows: result unused
                    bytes[a] = blk[k * 4];
                }
                const uint32_t xk[4][4] = {{xa0.x, xa1.x, xa0.y, xa1.y}, {xa0.z, xa1.z, xa0.w, xa1.w},
                                           {xb0.x, xb1.x, xb0.y, xb1.y}, {xb0.z, xb1.z, xb0.w, xb1.w}};
#pragma unroll
                for (int env = 0; env < EG; ++env) {
                    // s_in[env] of the group as bf16 pairs (hi, lo): lane l converts columns 2l, 2l+1,
                    // then every lane collects the 8 pairs of its 16 columns
                    uint32_t ph, pl;
                    {
                        const float2 sc = *reinterpret_cast<const float2 *>(slot + plan.off_scale +
                                                                            4 * (env * cwx + gcol + 2 * lane));
                        if (kHalf) split2h(sc.x, sc.y, ph, pl);
                        else split2(sc.x, sc.y, ph, pl);
                    }
                    uint32_t hA[4], hB[4], lA[4], lB[4];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        hA[p] = __shfl_sync(0xffffffffu, ph, 8 * q + p);
                        hB[p] = __shfl_sync(0xffffffffu, ph, 8 * q + 4 + p);
                        if (kLoPass) {
                            lA[p] = __shfl_sync(0xffffffffu, pl, 8 * q + p);
                            lB[p] = __shfl_sync(0xffffffffu, pl, 8 * q + 4 + p);
                        } else {
                            lA[p] = lB[p] = 0u;
                        }
                    }
                    // k-step outermost, rank blocks innermost: consecutive MMAs go to different
                    // accumulators, so none waits for the one before it
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint32_t h0 = (ks < 2) ? hA[2 * ks] : hB[2 * ks - 4], h1 = (ks < 2) ? hA[2 * ks + 1] : hB[2 * ks - 3];
                        const uint32_t l0 = (ks < 2) ? lA[2 * ks] : lB[2 * ks - 4], l1 = (ks < 2) ? lA[2 * ks + 1] : lB[2 * ks - 3];
#pragma unroll
                        for (int a = 0; a < R8; ++a) {
                            const uint32_t b = (ks < 2) ? (bytes[a] & 0xffu) : (bytes[a] >> 8);
                            const uint32_t m0 = pair_bits(b, 2 * (ks & 1)), m1 = pair_bits(b, 2 * (ks & 1) + 1);
                            if (!kHalf) {
                                mma_bf16(acc[env][0][a], xk[ks][0], xk[ks][1], xk[ks][2], xk[ks][3],
                                         with_signs(h0, m0), with_signs(h1, m1));
                                mma_bf16(acc[env][kSplitAcc ? 1 : 0][a], xk[ks][0], xk[ks][1], xk[ks][2], xk[ks][3],
                                         with_signs(l0, m0), with_signs(l1, m1));
                            } else if (kLoPass) {
                                mma_f16(acc[env][0][a], xk[ks][0], xk[ks][1], xk[ks][2], xk[ks][3],
                                        with_signs(h0, m0), with_signs(h1, m1));
                                mma_f16(acc[env][kSplitAcc ? 1 : 0][a], xk[ks][0], xk[ks][1], xk[ks][2], xk[ks][3],
                                        with_signs(l0, m0), with_signs(l1, m1));
                            } else {
                                // one pass: alternate k-steps between the two accumulator sets
                                mma_f16(acc[env][kSplitAcc ? (ks & 1) : 0][a], xk[ks][0], xk[ks][1], xk[ks][2], xk[ks][3],
                                        with_signs(h0, m0), with_signs(h1, m1));
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
            if (++s == S) { s = 0; sph ^= 1u; }
        }

        // ---- reduce u over the warps in a fixed order, z = s_r * u, split into bf16 hi + lo ---
#pragma unroll
        for (int env = 0; env < EG; ++env) {
#pragma unroll
            for (int a = 0; a < R8; ++a) {
                float c[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    c[e] = kSplitAcc ? acc[env][0][a][e] + acc[env][kSplitAcc ? 1 : 0][a][e] : acc[env][0][a][e];
                float *d0 = red + (((env * kConsumerWarps + warp) * kTile + g) * RP + 8 * a + 2 * q);
                *reinterpret_cast<float2 *>(d0) = make_float2(c[0], c[1]);
                *reinterpret_cast<float2 *>(d0 + 8 * RP) = make_float2(c[2], c[3]);
            }
        }
        consumer_sync<kConsumerThreads>();
        if (kClusters && xsplit > 1) {
            // This CTA's sums cover its share of d_in only.  Every pair of them goes to every CTA of
            // the cluster (its own included), followed by one arrival on that CTA's barrier; once
            // all CTAs have arrived here, the shares are added in the order of the CTAs' ranks.
            // A CTA whose own share is incomplete (a wait gave up) sends nothing: the others'
            // waits then give up too, and no CTA of the cluster writes to y.
            const bool whole = !*abort_flag;
            const uint32_t ux0 = sm_base + plan.off_ux;
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
                if (whole) {
                    const uint32_t off = (uint32_t)(((xrank * kTile + tok) * ZP + pr) * 8);
                    for (int dst = 0; dst < xsplit; ++dst) st_cluster_f2(mapa(ux0, dst) + off, u0, u1);
                }
            }
            // all of this CTA's stores, each thread's fenced at cluster scope, then the CTA barrier,
            // then one arrival per destination
            asm volatile("fence.acq_rel.cluster;" ::: "memory");
            consumer_sync<kConsumerThreads>();
            // (one thread per destination: an arrival with release is a round trip through the cluster)
            if (tid < xsplit && whole) mbar_arrive_remote(mapa(bar_ux, tid));
            const bool got = mbar_wait_cluster(wctx, bar_ux, 0u, kDevMmaWaitTimeout);
            const float *ux = reinterpret_cast<const float *>(smem + plan.off_ux);
            for (int idx = tid; idx < kTile * ZP; idx += kConsumerThreads) {
                const int tok = idx / ZP, pr = idx - tok * ZP;
                float u0 = 0.0f, u1 = 0.0f;
                for (int src = 0; src < xsplit && got; ++src) {
                    const float2 v = *reinterpret_cast<const float2 *>(ux + ((src * kTile + tok) * ZP + pr) * 2);
                    u0 += v.x;
                    u1 += v.y;
                }
                const int k = 2 * pr;
                const float z0 = (k < r) ? u0 * __ldg(P.s_r + k) : 0.0f;
                const float z1 = (k + 1 < r) ? u1 * __ldg(P.s_r + k + 1) : 0.0f;
                uint32_t hi, lo;
                split2(z0, z1, hi, lo);
                zH[idx] = hi;
                zL[idx] = lo;
            }
        } else
        for (int idx = tid; idx < EG * kTile * ZP; idx += kConsumerThreads) {
            const int env = idx / (kTile * ZP), rem = idx - env * (kTile * ZP);
            const int genv = grp * EG + env;           // envelope of the adapter
            if (genv >= ell) break;
            const int tok = rem / ZP, pr = rem - tok * ZP;
            float u0 = 0.0f, u1 = 0.0f;
            if (2 * pr < RP) {
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float2 v = *reinterpret_cast<const float2 *>(
                        red + (((env * kConsumerWarps + w) * kTile + tok) * RP + 2 * pr));
                    u0 += v.x;
                    u1 += v.y;
                }
            }
            const int k = 2 * pr;
            const float z0 = (k < r) ? u0 * __ldg(P.s_r + genv * r + k) : 0.0f;
            const float z1 = (k + 1 < r) ? u1 * __ldg(P.s_r + genv * r + k + 1) : 0.0f;
            uint32_t hi, lo;
            split2(z0, z1, hi, lo);
            zH[grp * (EG * kTile * ZP) + idx] = hi;
            zL[grp * (EG * kTile * ZP) + idx] = lo;
        }
        consumer_sync<kConsumerThreads>();
        }   // envelope groups

        // ---- second product: y[t,j] += s_out[j] sum_k B_sign[j,k] z[t,k] ---------------------
        // A fragments: k position (2q, 2q+1, 2q+8, 2q+9) of k-step s <-> ranks 16s + 4q + (0,1,2,3)
        // (with one envelope they are loaded once here, with several inside the item loop)
        auto load_z = [&](int env, uint32_t (&zh)[KS][4], uint32_t (&zl)[KS][4]) {
            const uint32_t *eh = zH + env * (kTile * ZP), *el = zL + env * (kTile * ZP);
#pragma unroll
            for (int s = 0; s < KS; ++s) {
                const uint2 h0 = *reinterpret_cast<const uint2 *>(eh + g * ZP + 8 * s + 2 * q);
                const uint2 h1 = *reinterpret_cast<const uint2 *>(eh + (g + 8) * ZP + 8 * s + 2 * q);
                const uint2 l0 = *reinterpret_cast<const uint2 *>(el + g * ZP + 8 * s + 2 * q);
                const uint2 l1 = *reinterpret_cast<const uint2 *>(el + (g + 8) * ZP + 8 * s + 2 * q);
                zh[s][0] = h0.x; zh[s][1] = h1.x; zh[s][2] = h0.y; zh[s][3] = h1.y;
                zl[s][0] = l0.x; zl[s][1] = l1.x; zl[s][2] = l0.y; zl[s][3] = l1.y;
            }
        };
        // z stays in registers across the items when all of it fits 16 of them: one envelope, or two
        // at rank <= 16 (then EG = 2 means exactly two envelopes)
        constexpr bool kZRes = (EGT == 2 && KS == 1);
        uint32_t zh[KS][4], zl[KS][4];
        uint32_t zh2[KS][4], zl2[KS][4];           // (second envelope; unused unless kZRes)
        if (ell == 1) load_z(0, zh, zl);
        if (kZRes) {
            load_z(0, zh, zl);
            load_z(1, zh2, zl2);
        }
        // A wait that gave up during the first product left u incomplete: this CTA then writes
        // nothing (its rows of y keep their old values) and only drains its items.
        const bool u_complete = !__any_sync(0xffffffffu, *abort_flag != 0);
        // (every thread that is going to write y has seen the previous kernel complete)
        if (prm.x_ready) asm volatile("griddepcontrol.wait;" ::: "memory");
        uint16_t *yrow0 = P.y + (t0 + g) * P.ldy;
        uint16_t *yrow1 = yrow0 + 8 * P.ldy;
        const bool vec32 = P.y_vec32 != 0;

        for (; it < n_items; ++it) {
            const bool ok = __all_sync(0xffffffffu, mbar_wait(wctx, bar_full(s), sph, kDevEpilogueWaitTimeout)) && u_complete;
            const int col0 = (yc_begin + (it - n_xi)) * cwy;
            const int cwv = (d_out - col0 < cwy) ? (d_out - col0) : cwy;
            if (gcol < cwv && ok) {
                const uint8_t *slot = smem + s * plan.slot_bytes;
                const uint8_t *bits = slot + plan.off_bits;
                // Output column of n-block i, accumulator column n = 2q + e: gcol + 16q + 2i + e, so
                // that a lane owns 16 consecutive columns.  As the holder of B-fragment column
                // n = g this lane expands the signs of j = gcol + 16(g>>1) + 2i + (g&1).
                const int jb = gcol + 16 * (g >> 1) + (g & 1);
                // the r sign bits of this lane's 8 B_sign rows, shifted so that k-step ks reads its
                // 4 bits at bit 16 ks
                typedef typename std::conditional<(RP > 32), uint64_t, uint32_t>::type bits_t;
                bits_t rb[8];
                if (RP == 16 && !GEN) {
                    // rows jb - (g&1) .. + 15 are 16 half-words: word i holds rows 2i (low) and 2i+1
                    const uint4 w0 = *reinterpret_cast<const uint4 *>(bits + 2 * (jb - (g & 1)));
                    const uint4 w1 = *reinterpret_cast<const uint4 *>(bits + 2 * (jb - (g & 1)) + 16);
                    const uint32_t w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
                    const int sh = 16 * (g & 1) + 4 * q;
#pragma unroll
                    for (int i = 0; i < 8; ++i) rb[i] = (bits_t)(w[i] >> sh);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) rb[i] = (bits_t)(b_row_bits<RP, GEN>(bits, jb + 2 * i, r) >> (4 * q));
                }
                // The lane's 16 columns are done as two halves of 8 (n-blocks 4cc .. 4cc+3) to keep
                // the live registers low; the results of both halves leave in one 256-bit store.
                uint32_t out[2][8];
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    float vs[2][8];                                  // y + sum over the envelopes of s_out * v
#pragma unroll
                    for (int half = 0; half < 2; ++half) {              // token rows g and g + 8
                        const uint4 yv = *reinterpret_cast<const uint4 *>(slot + (half == 0 ? off_r0 : off_r1) +
                                                                           (cc == 0 ? pc0 : pc1));
                        const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            if (kHalf) {
                                const float2 f = unpack2h(yw[i]);
                                vs[half][2 * i] = f.x;
                                vs[half][2 * i + 1] = f.y;
                            } else {
                                vs[half][2 * i] = lo_f(yw[i]);
                                vs[half][2 * i + 1] = hi_f(yw[i]);
                            }
                        }
                    }
                    // the envelopes in runs of EG whose bodies are unrolled (a single run when all of
                    // them fit one pass of the first product)
                    for (int eb = 0; eb < ell; eb += EG)
#pragma unroll
                    for (int ei = 0; ei < EG; ++ei) {
                        const int env = eb + ei;
                        if (EGT != 1 && env >= ell) break;
                        if (EGT != 1 && !kZRes) load_z(env, zh, zl);
                        // (resident z: envelope 0 in zh / zl, envelope 1 in zh2 / zl2)
                        const uint32_t (*azh)[4] = (kZRes && ei == 1) ? zh2 : zh;
                        const uint32_t (*azl)[4] = (kZRes && ei == 1) ? zl2 : zl;
                        float c[4][4];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int e = 0; e < 4; ++e) c[i][e] = 0.0f;
                        // k-step outermost, n-blocks innermost: consecutive MMAs go to different accumulators
#pragma unroll
                        for (int ks = 0; ks < KS; ++ks) {
                            uint32_t b0[4], b1[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const uint32_t nib = (uint32_t)(rb[4 * cc + i] >> (16 * ks)) & 0xfu;
                                b0[i] = with_signs(0x3f803f80u, nib * 0x40008000u);
                                b1[i] = with_signs(0x3f803f80u, nib * 0x10002000u);
                            }
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                mma_bf16(c[i], azh[ks][0], azh[ks][1], azh[ks][2], azh[ks][3], b0[i], b1[i]);
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                mma_bf16(c[i], azl[ks][0], azl[ks][1], azl[ks][2], azl[ks][3], b0[i], b1[i]);
                        }
                        const float4 *so4 = reinterpret_cast<const float4 *>(
                            slot + plan.off_scale + 4 * (env * cwy + gcol + 16 * q + 8 * cc));
                        const float4 s0 = so4[0], s1 = so4[1];
                        const float so[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
                        for (int half = 0; half < 2; ++half)
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                if (EGT != 1) {
                                    // several envelopes: the packed form was measured ahead (7 % at two envelopes)
                                    fma2(vs[half][2 * i], vs[half][2 * i + 1], so[2 * i], so[2 * i + 1], c[i][2 * half], c[i][2 * half + 1]);
                                } else {
                                    vs[half][2 * i] = fmaf(so[2 * i], c[i][2 * half], vs[half][2 * i]);
                                    vs[half][2 * i + 1] = fmaf(so[2 * i + 1], c[i][2 * half + 1], vs[half][2 * i + 1]);
                                }
                            }
                    }
#pragma unroll
                    for (int half = 0; half < 2; ++half)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            out[half][4 * cc + i] = kHalf ? pack2h(vs[half][2 * i], vs[half][2 * i + 1])
                                                          : pack2(vs[half][2 * i], vs[half][2 * i + 1]);
                }
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (half == 0 ? v0 : v1) {
                        uint16_t *dst = (half == 0 ? yrow0 : yrow1) + col0 + gcol + 16 * q;
                        const uint32_t oa[4] = {out[half][0], out[half][1], out[half][2], out[half][3]};
                        const uint32_t ob[4] = {out[half][4], out[half][5], out[half][6], out[half][7]};
                        if (vec32) {
                            st_global_256(dst, oa, ob);
                        } else {
                            __stcs(reinterpret_cast<uint4 *>(dst), make_uint4(oa[0], oa[1], oa[2], oa[3]));
                            __stcs(reinterpret_cast<uint4 *>(dst) + 1, make_uint4(ob[0], ob[1], ob[2], ob[3]));
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
            if (++s == S) { s = 0; sph ^= 1u; }
        }
    }

    // ---- teardown: after an abort, give copies that may still be in flight time to land ---------
    __syncthreads();
    if (*abort_flag) {
        const long long start = clock64();
        while (clock64() - start < 2000000LL) __nanosleep(1000);
    }
    if (!prm.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ------------------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

bool encode(CUtensorMap *map, CUtensorMapDataType type, int rank, const void *base, const cuuint64_t *dims,
            const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swizzle)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, type, (cuuint32_t)rank, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major T x d matrix of 16-bit elements (bf16 or half: the map only moves them; row pitch ld
// elements, d % 64 == 0) seen as the 3-D tensor
// (column in group: 64, row: T, column group: d / 64); a box is 64 x 16 rows x `groups`.
bool make_data_map(CUtensorMap *map, const void *base, int64_t T, int64_t d, int64_t ld, int groups)
{
    const cuuint64_t dims[3] = {(cuuint64_t)kGroup, (cuuint64_t)T, (cuuint64_t)(d / kGroup)};
    const cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)kGroup * 2};
    const cuuint32_t box[3] = {(cuuint32_t)kGroup, (cuuint32_t)kTile, (cuuint32_t)groups};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// A dense array seen as n_rows rows of `row_elems` 4-byte elements; a box is `box_rows` whole
// rows, laid out densely in shared memory.
bool make_linear_map(CUtensorMap *map, CUtensorMapDataType type, const void *base, int row_elems,
                     int64_t n_rows, int box_rows)
{
    const cuuint64_t dims[2] = {(cuuint64_t)row_elems, (cuuint64_t)n_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_elems * 4};
    const cuuint32_t box[2] = {(cuuint32_t)row_elems, (cuuint32_t)box_rows};
    return encode(map, type, 2, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE);
}

// ell x d float32 scales (envelope e in row e, d % 64 == 0) seen as (64, d / 64, ell); a box is
// `groups` groups of `box_ell` envelopes: it lands as [envelope][group][64 floats] (envelopes past
// the adapter's last one are filled with zeros).
bool make_scale_map(CUtensorMap *map, const float *base, int64_t d, int ell, int box_ell, int groups)
{
    const cuuint64_t dims[3] = {(cuuint64_t)kGroup, (cuuint64_t)(d / kGroup), (cuuint64_t)ell};
    const cuuint64_t strides[2] = {(cuuint64_t)kGroup * 4, (cuuint64_t)d * 4};
    const cuuint32_t box[3] = {(cuuint32_t)kGroup, (cuuint32_t)groups, (cuuint32_t)box_ell};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE);
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

// The kernel instantiation for a launch, with its dynamic shared-memory limit raised once.
template <int RP, int NW, int EG, int IO, bool GEN>
const void *kernel_one()
{
    static std::once_flag once;
    static cudaError_t attr_rc = cudaSuccess;
    std::call_once(once, []() {
        attr_rc = cudaFuncSetAttribute(mma_forward_kernel<RP, NW, EG, IO, GEN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kSmemBudget);
    });
    if (attr_rc != cudaSuccess) return nullptr;
    return reinterpret_cast<const void *>(&mma_forward_kernel<RP, NW, EG, IO, GEN>);
}

// Envelopes per pass of the first product (the kernel's EGT): as many as fit 64 partial sums per
// token row (EG * RP <= 64), a power of two.
int envelopes_per_pass(int rp, int ell)
{
    const int cap = kMaxRank / rp;
    int eg = 1;
    while (eg < ell && eg < cap) eg *= 2;
    return (eg == 1 && ell > 1) ? 0 : eg;       // 0: one per pass, several in all (see the kernel)
}

template <int NW, int IO, bool GEN>
const void *kernel_rank(int rp, int eg)
{
    switch (rp * 16 + eg) {
        case 8 * 16 + 1:  return kernel_one<8, NW, 1, IO, GEN>();
        case 8 * 16 + 2:  return kernel_one<8, NW, 2, IO, GEN>();
        case 8 * 16 + 4:  return kernel_one<8, NW, 4, IO, GEN>();
        case 8 * 16 + 8:  return kernel_one<8, NW, 8, IO, GEN>();
        case 16 * 16 + 1: return kernel_one<16, NW, 1, IO, GEN>();
        case 16 * 16 + 2: return kernel_one<16, NW, 2, IO, GEN>();
        case 16 * 16 + 4: return kernel_one<16, NW, 4, IO, GEN>();
        case 32 * 16 + 1: return kernel_one<32, NW, 1, IO, GEN>();
        case 32 * 16 + 2: return kernel_one<32, NW, 2, IO, GEN>();
        case 64 * 16 + 1: return kernel_one<64, NW, 1, IO, GEN>();
        case 64 * 16 + 0: return kernel_one<64, NW, 0, IO, GEN>();
        default: break;
    }
    // single envelope, CTAs sharing the first product as clusters: small CTAs only
    if (NW == 8 && eg == -1) {
        switch (rp) {
            case 8:  return kernel_one<8, 8, -1, IO, GEN>();
            case 16: return kernel_one<16, 8, -1, IO, GEN>();
            case 32: return kernel_one<32, 8, -1, IO, GEN>();
            case 64: return kernel_one<64, 8, -1, IO, GEN>();
            default: break;
        }
    }
    return nullptr;
}

template <int IO>
const void *kernel_io(int rp, int nw, int eg, bool gen)
{
    if (gen)       // ranks other than 8 / 16 / 32 / 64, in instantiations of their own
        return nw == kMaxWarps ? kernel_rank<kMaxWarps, IO, true>(rp, eg) : kernel_rank<8, IO, true>(rp, eg);
    return nw == kMaxWarps ? kernel_rank<kMaxWarps, IO, false>(rp, eg) : kernel_rank<8, IO, false>(rp, eg);
}

}  // namespace

bool mma_supported(const lordba_proj &p, int64_t T, int dtype)
{
    if ((dtype != LORDBA_BF16 && dtype != LORDBA_F16) || T < 1 || T > (1 << 30)) return false;
    const int ell = ((p.flags >> 8) & 0xf) + 1;
    if (ell > LORDBA_MAX_ELL || p.r < 1 || p.r > kMaxRank) return false;
    // a carrier is copied as whole 64-byte rows of sign bytes
    if ((p.d_in * p.r) % 512 != 0 || (p.d_out * p.r) % 512 != 0) return false;
    // whole 64-column groups (the 3-D tensor view), 16-byte aligned rows
    if (p.d_in % kGroup != 0 || p.d_out % kGroup != 0 || p.ldx % 8 != 0 || p.ldy % 8 != 0) return false;
    if (p.d_in > (1 << 30) || p.d_out > (1 << 30)) return false;
    if (reinterpret_cast<uintptr_t>(p.x) % 16 || reinterpret_cast<uintptr_t>(p.y) % 16) return false;
    // the scale and carrier slices of an item travel as bulk copies: 16-byte aligned sources
    if (reinterpret_cast<uintptr_t>(p.s_in) % 16 || reinterpret_cast<uintptr_t>(p.s_out) % 16 ||
        reinterpret_cast<uintptr_t>(p.packed_A) % 16 || reinterpret_cast<uintptr_t>(p.packed_B) % 16)
        return false;
    return encode_fn() != nullptr;
}

int launch_forward_mma(const lordba_proj *projs, const int64_t *tokens, int64_t T, int n, const FamilySelector &fsel,
                       LaunchSink &sink, bool batch_checked, int *launches)
{
    if (n == 0) return LORDBA_OK;
    const int dtype = fsel.dtype;
    if (dtype != LORDBA_BF16 && dtype != LORDBA_F16) return LORDBA_OK;     // float32: the FMA kernel's
    int *status = nullptr;
    const int sms = sm_count();
    bool all_overlap = true;          // the caller's promise covers the call only if every projection carries it
    for (int i = 0; i < n; ++i) all_overlap = all_overlap && (projs[i].flags & LORDBA_PROJ_OVERLAP);
    // one launch per (element / scale kind, envelopes, padded rank) present in the call, up to
    // kMaxBatch projections each; the key of every projection is worked out once
    auto io_of = [&](const lordba_proj &q) {
        if (dtype == LORDBA_BF16) return (int)kIoBf16;
        return (q.flags & LORDBA_PROJ_SCALES_F16) ? (int)kIoF16Exact : (int)kIoF16;
    };
    auto key_of = [](int io, int ell, int gen, int rp) { return (uint16_t)(((io * 9 + ell) * 2 + gen) * 128 + rp); };
    uint16_t keys[kMaxCallProjs];
    uint32_t ell_seen = 0;
    for (int i = 0; i < n; ++i) {
        const int64_t rows_i = rows_of(tokens, T, i);
        keys[i] = 0xffffu;
        if (rows_i <= 0 || fsel.family(projs[i], rows_i) != LORDBA_VARIANT_MMA) continue;
        const int rp_i = padded_rank(projs[i].r), ell_i = ((projs[i].flags >> 8) & 0xf) + 1;
        keys[i] = key_of(io_of(projs[i]), ell_i, projs[i].r != rp_i ? 1 : 0, rp_i);
        ell_seen |= 1u << ell_i;
    }
    const int io_first = (dtype == LORDBA_BF16) ? kIoBf16 : kIoF16;
    const int io_last = (dtype == LORDBA_BF16) ? kIoBf16 : kIoF16Exact;
    for (int io = io_first; io <= io_last; ++io)
    for (int ell = 1; ell <= LORDBA_MAX_ELL; ++ell)
    for (int gen = 0; gen <= 1; ++gen)
    for (int rp = 8; rp <= kMaxRank; rp *= 2) {
        if (!(ell_seen & (1u << ell))) continue;
        const uint16_t key = key_of(io, ell, gen, rp);
        const int egt = envelopes_per_pass(rp, ell);
        const int eg = egt == 0 ? 1 : egt;
        const lordba_proj *sel[kMaxBatch];
        int64_t sel_T[kMaxBatch];
        int m = 0, max_r = 0, min_cw = 128;
        int64_t min_dout = (int64_t)1 << 40;
        for (int i = 0; i <= n; ++i) {
            const bool take = (i < n) && keys[i] == key;
            if (take) {
                sel_T[m] = rows_of(tokens, T, i);
                sel[m++] = &projs[i];
                if (projs[i].r > max_r) max_r = projs[i].r;
                // narrowest y item of this projection: its sign bytes must be whole 64-byte rows
                const int need_cw = (projs[i].r % 4 == 0) ? 128 : (projs[i].r % 2 == 0) ? 256 : 512;
                if (need_cw > min_cw) min_cw = need_cw;
                if (projs[i].d_out < min_dout) min_dout = projs[i].d_out;
            }
            if (m == kMaxBatch || (i == n && m > 0)) {
                if (!status && !(status = device_status_word())) return LORDBA_ECUDA;
                // CTAs start in grid order (all tiles of projection 0, then of projection 1, ...):
                // projections with the most bytes per token go first, so that the last, partly
                // filled wave consists of the cheapest tiles (stable insertion sort).
                for (int a = 1; a < m; ++a) {
                    const lordba_proj *pa = sel[a];
                    const int64_t ta = sel_T[a], ka = pa->d_in + 2 * pa->d_out;
                    int b = a - 1;
                    while (b >= 0 && sel[b]->d_in + 2 * sel[b]->d_out < ka) {
                        sel[b + 1] = sel[b]; sel_T[b + 1] = sel_T[b];
                        --b;
                    }
                    sel[b + 1] = pa; sel_T[b + 1] = ta;
                }
                // Tile height: always the full 16 rows of an MMA tile.  Shorter tiles that spread a
                // call evenly over whole waves of SMs (14 rows for T = 2048) were measured slower at
                // every size from 8 to 4096 tokens: an MMA costs the same with 14 or 16 live rows,
                // and fewer, fuller CTAs leave room for the neighbouring calls' CTAs.
                const int64_t rows = kTile;
                const bool overlaps_neighbours = (*launches == 0) ? all_overlap : batch_checked;
                // the first launch of a call that waits for its predecessor may still start on x
                bool x_ready = !overlaps_neighbours && *launches == 0;
                for (int k = 0; k < m; ++k) x_ready = x_ready && (sel[k]->flags & LORDBA_PROJ_X_READY);
                int64_t tiles = 0, all_tiles = 0;      // widest projection (grid.x), and the sum
                for (int k = 0; k < m; ++k) {
                    const int64_t tk = (sel_T[k] + rows - 1) / rows;
                    all_tiles += tk;
                    if (tk > tiles) tiles = tk;
                }
                // Few tokens: split the y items over several CTAs per tile (each repeats the
                // first product), with narrower items so that there is something to split.
                int64_t want_splits = sms / all_tiles;
                if (want_splits < 1) want_splits = 1;
                // Two small CTAs per SM when there is a second CTA to pair with: more than one
                // wave of tiles, or a call that may overlap its neighbours.  One's start-up and
                // first-load latency then hide behind the other's streaming.  A lone single-wave
                // call keeps one CTA with 16 consumer warps per SM.
                // Few tiles of a single-envelope launch (a decode-sized call, a short prompt): the CTAs
                // that split a tile's y items also share its first product, as clusters of 4 or 8 along
                // grid z.  Each CTA streams its part of d_in only and the partial sums go round the
                // cluster, instead of every CTA repeating the product over all of d_in, which was most
                // of such a call's time (layer at 1 to 8 tokens: 11.3 -> 5.8 us per call that waits
                // for its predecessor; a 4096-wide projection alone at 8 to 256 tokens 5.9 - 6.7 ->
                // 4.5 - 5.6 us).  Small CTAs (512-column items), one per SM.  Only with room for at
                // least 4 CTAs per tile: clusters of 2 measured behind the repeated product
                // (layer at 128 tokens, waiting: 13.6 against 12.8 us).
                int xsplit = 1;
                int64_t max_din = 0;
                for (int k = 0; k < m; ++k)
                    if (sel[k]->d_in > max_din) max_din = sel[k]->d_in;
                if (egt == 1 && max_din >= 4 * 8 * kGroup) {
                    const int64_t room = sms / all_tiles;
                    xsplit = room >= 8 ? 8 : room >= 4 ? 4 : 1;
                    if (xsplit > 1) want_splits = room / xsplit * xsplit;
                }
                const int nw = (all_tiles > sms || overlaps_neighbours || xsplit > 1) ? 8 : kMaxWarps;
                const int max_chunk = nw * kGroup;
                const int smem_budget = (nw == kMaxWarps) ? kSmemBudget : kSmemBudgetHalf;
                int cw = max_chunk;
                int64_t splits;
                if (xsplit > 1) {
                    // the widest items with which no CTA of the launch gets more y items than it must
                    // (an item costs about the same time whatever its width)
                    splits = want_splits > 64 ? 64 : want_splits;
                    auto y_items = [&](int w) {
                        int64_t worst = 0;
                        for (int k = 0; k < m; ++k) {
                            const int64_t c = ((sel[k]->d_out + w - 1) / w + splits - 1) / splits;
                            if (c > worst) worst = c;
                        }
                        return worst;
                    };
                    for (int w = max_chunk / 2; w >= min_cw; w /= 2)
                        if (y_items(w) < y_items(cw)) cw = w;
                } else {
                    while (cw > min_cw && (min_dout + cw - 1) / cw < want_splits) cw /= 2;
                    splits = (min_dout + cw - 1) / cw;
                    if (splits > want_splits) splits = want_splits;
                    if (splits > 64) splits = 64;
                }

                MmaBatch b;
                std::memset(&b, 0, sizeof(b));
                for (int k = 0; k < m; ++k) {
                    const lordba_proj &q = *sel[k];
                    MmaProj &t = b.p[k];
                    // sign bytes: d r / 8 per carrier, as rows of 16 words; an item holds cw r / 512 rows
                    if (!make_data_map(&t.x_map, q.x, sel_T[k], q.d_in, q.ldx, nw) ||
                        !make_data_map(&t.y_map, q.y, sel_T[k], q.d_out, q.ldy, cw / kGroup) ||
                        !make_scale_map(&t.si_map, q.s_in, q.d_in, ell, eg, nw) ||
                        !make_scale_map(&t.so_map, q.s_out, q.d_out, ell, ell, cw / kGroup) ||
                        !make_linear_map(&t.pa_map, CU_TENSOR_MAP_DATA_TYPE_UINT32, q.packed_A, 16,
                                         q.d_in * q.r / 512, max_chunk * q.r / 512) ||
                        !make_linear_map(&t.pb_map, CU_TENSOR_MAP_DATA_TYPE_UINT32, q.packed_B, 16,
                                         q.d_out * q.r / 512, cw * q.r / 512))
                        return LORDBA_ECUDA;
                    t.s_r = q.s_r;
                    t.y = static_cast<uint16_t *>(q.y);
                    t.ldy = q.ldy;
                    t.T = sel_T[k];
                    t.d_in = (int)q.d_in; t.d_out = (int)q.d_out; t.r = q.r;
                    t.y_vec32 = (reinterpret_cast<uintptr_t>(q.y) % 32 == 0 && q.ldy % 16 == 0) ? 1 : 0;
                }
                MmaParams prm;
                std::memset(&prm, 0, sizeof(prm));
                prm.rows = (int)rows; prm.cwy = cw; prm.status = status;
                prm.wait_prev = !overlaps_neighbours;
                prm.x_ready = x_ready;
                prm.xsplit = xsplit;
                prm.spread_issue = xsplit > 1 ? 1 : 0;
                prm.skip_item = test_skip_item();
                prm.gate_y = (prm.wait_prev && xsplit == 1) ? 2 : 0;   // (measured: a call that waits for its predecessor, 12.1 -> 11.8 us; later items lose it again)
                prm.ell = ell;
                ++*launches;
                int slots = kMaxSlots;
                while (slots > 2 && make_plan(nw, rp, max_r, slots, eg, ell, cw, xsplit).total > smem_budget) --slots;
                const SmemPlan plan = make_plan(nw, rp, max_r, slots, eg, ell, cw, xsplit);
                if (plan.total > kSmemBudget) return LORDBA_ECUDA;
                prm.slots = slots;
                LaunchRec rec;
                std::memset(&rec, 0, sizeof(rec));
                const int inst = xsplit > 1 ? -1 : egt;      // (the instantiation with the cluster exchange)
                rec.func = io == kIoBf16 ? kernel_io<kIoBf16>(rp, nw, inst, gen != 0)
                           : io == kIoF16 ? kernel_io<kIoF16>(rp, nw, inst, gen != 0)
                                          : kernel_io<kIoF16Exact>(rp, nw, inst, gen != 0);
                if (!rec.func) return LORDBA_ECUDA;
                rec.grid[0] = (unsigned)tiles; rec.grid[1] = (unsigned)m; rec.grid[2] = (unsigned)splits;
                rec.block = nw * 32 + 32;
                rec.smem = (uint32_t)plan.total;
                // Programmatic dependent launch: the CTAs of this grid may become resident, fetch their
                // parameters and set up their barriers while the previous kernel of the stream drains; they
                // touch no global data before griddepcontrol.wait, which returns once that kernel has
                // completed and its writes are visible.
                rec.pdl = 1;
                rec.cluster = xsplit > 1 ? (uint32_t)xsplit : 0;
                rec.cluster_z = xsplit > 1 ? 1 : 0;
                rec.n_args = 2;
                rec.arg_bytes[0] = sizeof(MmaBatch);
                rec.arg_bytes[1] = sizeof(MmaParams);
                const int rc = sink.emit(rec, &b, &prm);
                if (rc != LORDBA_OK) return rc;
                m = 0; max_r = 0; min_cw = 128; min_dout = (int64_t)1 << 40;
            }
        }
    }
    return LORDBA_OK;
}

}  // namespace lordba
