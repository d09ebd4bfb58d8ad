// Tensor-core kernel of the LoRDBA adapter forward (bf16 or float16 activations), sm_100a:
//
//   y[t,:] += s_out * ( B_sign ( s_r * ( A_sign ( s_in * x[t,:] ) ) ) )        (Eq. 8 / Eq. 9)
//
// Work unit: one tile of 128 tokens, handled by a thread-block cluster of C
// CTAs (C = 1, 2, 4 or 8).  CTA c of the cluster streams its share of the d_in
// axis for the first binary product and its share of the d_out axis for the
// second one; the 128 x r intermediate is combined across the cluster through
// distributed shared memory and never leaves the chip.  Per CTA:
//
//   warp 0      TMA producer: 128 x 64 bf16 boxes of x, then of y, into a ring of
//               128B-swizzled shared-memory slots (cp.async.bulk.tensor, mbarrier tx).
//   warps 2-9   operand generators (two groups of four warps on alternate chunks):
//               expand packed sign bits into bf16 MMA operands in a ring of their own.  Stage 1: W1[k,i] = A_sign[k,i]*s_in[i] as a
//               hi/lo bf16 pair (rows 0..r-1 hi, r..2r-1 lo) so that s_in keeps
//               ~16 mantissa bits.  Stage 2: W2[j,k] = B_sign[j,k] (+-1, exact).
//   warp 1      MMA issuer (one thread): tcgen05.mma kind::f16, M=128.
//               Stage 1: U[128 x 2r] += X[128 x 64] * W1^T, accumulated in TMEM
//               over the CTA's K chunks.  Stage 2, per 64 output columns:
//               V[128 x 64] = Zhi * W2^T + Zlo * W2^T (z split hi/lo as well).
//   warps 10-17 epilogue: TMEM -> registers.  After stage 1: u = U_hi + U_lo; with
//               a cluster the partial sums are pushed to the CTA that owns the row,
//               reduced there in a fixed order, scaled by s_r, split into bf16
//               hi/lo and pushed back into every CTA's stage-2 operand buffer; a
//               lone CTA writes z = s_r * u straight into its own buffer.
//               After stage 2 (two groups of four warps on alternate chunks): y
//               tile (already in the slot) += s_out * V in fp32, rounded once to
//               bf16 in place, TMA-stored from the same slot.
//
// Two-envelope adapters (Def. 1 / Eq. 4, ell = 2, ell * r <= 64) run in the instantiation L = 2:
// both envelopes use the same carriers, so W1 carries every sign under each envelope's s_in
// (rows e r + k hi, ell r + e r + k lo) and U has 2 ell r columns; z is one hi/lo operand pair per
// envelope; stage 2 runs per envelope over the same W2 into ell accumulators, and the epilogue
// adds s_out[e] * V_e over the envelopes before the one rounding.
//
// The roles are decoupled by mbarriers only, so each one's per-chunk latency is
// a ceiling for the whole pipeline; the single MMA-issuing thread in particular
// carries its ring positions and descriptor words instead of recomputing them.
// Consecutive launches of one batched call overlap through programmatic
// dependent launch (B.wait_prev = 0 for all but the first).
//
// Every mbarrier wait is bounded: after ~1 s it records a code in the device
// status word, raises the CTA's abort flag (all later waits return at once) and
// the kernel runs to its normal teardown, which frees TMEM.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstring>
#include <mutex>

#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kTileM = 128;             // MMA M = TMEM lanes; a tile holds tile_rows <= 128 tokens
constexpr int kChunk = 64;              // columns per TMA box (128 bytes of bf16)
constexpr int kGenGroupThreads = 128;      // one generator group: four warps
constexpr int kGenGroups = 2;             // the groups take alternate chunks, so two operands are in the making
constexpr int kGenThreads = kGenGroups * kGenGroupThreads;   // warps 2-9
constexpr int kEpiThreads = 256;          // warps 10-17
constexpr int kThreads = 64 + kGenThreads + kEpiThreads;
constexpr int kMaxTcBatch = 96;          // 96 x 320 bytes of descriptors: inside the 32 KiB of kernel parameters
constexpr int kMaxTcEll = 2;            // envelopes per adapter this kernel takes (ell * r <= kMaxRank)
constexpr int kTmemU = 0;               // stage-1 accumulator columns [0, 2 ell r)
constexpr int kTmemV = 128;             // stage-2 accumulators: two buffers of ell x 64 columns
__host__ __device__ inline uint32_t tmem_cols(int ell) { return ell > 1 ? 512u : 256u; }
constexpr int kSmemBudget = 227 * 1024;

// Element type of x and y, and how s_in enters the first product (same meaning as in the
// streaming kernel).
enum IoKind {
    kIoBf16 = 0,      // bfloat16; W1 = +-s_in as bf16 hi rows and lo rows (N = 2r)
    kIoF16 = 1,       // IEEE half; W1 as half hi rows and lo rows (N = 2r)
    kIoF16Exact = 2   // IEEE half; s_in stated to be exact in half precision: hi rows only (N = r)
};

struct alignas(64) TcProj {
    CUtensorMap x_map;
    CUtensorMap y_map;
    const uint32_t *packed_A;
    const uint32_t *packed_B;
    const float *s_in;
    const float *s_r;
    const float *s_out;
    int d_in, d_out;
    int nk, nn;            // 64-column chunks of d_in / d_out
    int tile_start;        // index of this projection's first tile among the launch's tiles
};

struct TcBatch {
    TcProj p[kMaxTcBatch];
    int n_proj;
    int total_tiles;       // projections may differ in their token counts (tile_start of each)
    int r;                 // rank, multiple of 8
    int ell;               // envelopes per adapter (1 or 2): scale triples that share the carriers
    int kp;                // r rounded up to 16 (K extent of the stage-2 MMA)
    int cluster;           // CTAs per cluster
    int slots;             // ring depth
    int tile_rows;         // tokens per tile (multiple of cluster, <= 128); rows above it are padding
    int io;                // element type of x / y and form of s_in: see IoKind
    int wait_prev;         // 1: the previous kernel of the stream must be complete before any global access
    int skip_item;         // -1; the test-hooks build can name one chunk whose copy requests are left out
    int *status;
};

// ---- shared-memory plan (offsets from a 1024-byte aligned base), same on host and device ----
constexpr int kOps = 3;    // operand buffers (generated W1 / W2 tiles), a ring of their own

struct SmemPlan {
    int slot_data;          // bytes reserved for the x / y box of a slot (multiple of 1024)
    int slot_stride;        // + the slot's raw scale values and sign bytes
    int op_bytes, off_ops;  // one generated operand tile; start of the operand ring
    int off_z, z_bytes;     // per envelope: z hi tile, then z lo tile
    int raw_sign;           // offset of the sign bytes in a slot's raw area (behind the scale rows)
    int off_rx, off_bar, off_misc, total;
};

__host__ __device__ inline int round_up(int a, int b) { return (a + b - 1) / b * b; }

__host__ __device__ inline int aux_operand_bytes(int r, int kp, int ell)
{
    const int w1 = 2 * ell * r * 128;        // 2 ell r rows x 64 bf16
    const int w2 = kChunk * kp * 2;          // 64 rows x kp bf16
    return w1 > w2 ? w1 : w2;
}

__host__ __device__ inline SmemPlan make_plan(int r, int kp, int slots, int tile_rows, int cluster, int ell)
{
    SmemPlan s;
    // The MMA reads 128 rows (16 KiB) from the start of a slot whatever tile_rows is; what lies
    // beyond the box (this slot's raw area, the next slot) only reaches accumulator rows that
    // nobody reads.  `total` is padded so that this read stays inside the allocation.
    s.slot_data = round_up(tile_rows * kChunk * 2, 1024);
    // behind the box: 256 B of raw scale values per envelope and up to 512 B of raw sign bytes
    // (8 r bytes; ell * r <= kMaxRank)
    s.raw_sign = 256 * ell;
    s.slot_stride = s.slot_data + round_up(s.raw_sign + 8 * r, 1024);
    // The generated operands live in a short ring of their own (the MMA is done with one within
    // a microsecond), so that the data ring can be deep enough to cover the load latency at
    // any rank.
    s.op_bytes = round_up(aux_operand_bytes(r, kp, ell), 1024);
    s.off_ops = slots * s.slot_stride;
    s.z_bytes = (kTileM / 8) * (kp / 8) * 128;
    s.off_z = s.off_ops + kOps * s.op_bytes;
    s.off_rx = s.off_z + 2 * ell * s.z_bytes;
    // the exchange buffer for partial u exists only when a cluster splits the feature axes
    s.off_bar = s.off_rx + (cluster > 1 ? kTileM * ell * r * 4 : 0);
    s.off_misc = s.off_bar + (3 * slots + 2 * kOps + 8) * 8;
    s.total = s.off_misc + 16;
    const int last_read_end = (slots - 1) * s.slot_stride + kTileM * kChunk * 2;
    if (s.total < last_read_end) s.total = last_read_end;
    return s;
}

// ---------------------------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t v; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(v)); return v;
}
__device__ __forceinline__ uint32_t cluster_id_x()
{
    uint32_t v; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(v)); return v;
}
__device__ __forceinline__ uint32_t n_cluster_id_x()
{
    uint32_t v; asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(v)); return v;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank)
{
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
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
// arrive on a barrier of any CTA of the cluster (address from mapa), release at cluster scope
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\n"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                 "selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\n"
                 "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
                 "selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}

struct WaitCtx {
    volatile int *abort_flag;   // shared memory
    int *status;                // global status word
};

// Bounded wait.  Returns false once the CTA has given up.
template <bool kClusterScope>
__device__ __forceinline__ bool mbar_wait(const WaitCtx &w, uint32_t bar, uint32_t parity, int code)
{
    // fast path first: the abort flag is looked at only when the phase is not complete yet (after
    // an abort some barriers never complete, and the loop below then returns within 64 polls)
    if (kClusterScope ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if (*w.abort_flag) return false;
    const long long start = clock64();
    uint32_t spins = 0;
    for (;;) {
        if (kClusterScope ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
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

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// plain (untiled) bulk copy global -> shared; both addresses 16-byte aligned, size a multiple of 16
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Shared-memory matrix descriptor (tcgen05), 64 bits: start address >> 4 in bits 0..13, leading
// byte offset >> 4 in bits 16..29, stride byte offset >> 4 in bits 32..45, descriptor version 1 at
// bit 46, layout type in bits 61..63 (0 = no swizzle, 2 = 128B swizzle).  The MMA issuer builds the
// two 32-bit words itself.

// Instruction descriptor, kind::f16: D = fp32, A and B both bf16 (format 1) or both half (format
// 0; the two never differ), both K-major, M x N tile.
__device__ __forceinline__ uint32_t instr_desc(int m, int n, bool half_operands)
{
    const uint32_t fmt = half_operands ? 0u : ((1u << 7) | (1u << 10));
    return (1u << 4) | fmt | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// tcgen05.mma with the descriptors as (low, high) words: the issuing thread keeps the high words
// and the base of the low words in registers and only adds a 16-byte-unit offset per MMA.
__device__ __forceinline__ void mma_bf16_words(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                               uint32_t b_hi, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n.reg .pred p;\n.reg .b64 da, db;\nsetp.ne.b32 p, %6, 0;\n"
                 "mov.b64 da, {%1, %2};\nmov.b64 db, {%3, %4};\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float v[8])
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t r[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t r[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void st_cluster_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
__device__ __forceinline__ uint32_t pack2_f16(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ float2 unpack2_f16(uint32_t w) { return __half22float2(*reinterpret_cast<const __half2 *>(&w)); }

// 8 sign bits (bit 1 = +1) -> XOR masks over four bf16 pairs (a 0 bit flips the sign).  b times
// (2^(15-2p) + 2^(30-2p)) is two disjoint shifted copies of the byte that put bit 2p at position
// 15 and bit 2p+1 at position 31; only those two positions are kept, inverted.  No table: the
// shared-memory pipe is the busiest unit of this kernel.
__device__ __forceinline__ uint4 sign_masks(uint32_t b)
{
    uint4 m;
    m.x = ~(b * ((1u << 15) + (1u << 30))) & 0x80008000u;
    m.y = ~(b * ((1u << 13) + (1u << 28))) & 0x80008000u;
    m.z = ~(b * ((1u << 11) + (1u << 26))) & 0x80008000u;
    m.w = ~(b * ((1u << 9) + (1u << 24))) & 0x80008000u;
    return m;
}

// Slot of the data ring and phase of its barriers for chunk counter `it`: set once per tile (one
// division), then stepped, so that no role divides per chunk.
struct RingPos {
    int s;
    uint32_t ph;
    __device__ __forceinline__ void set(uint32_t it, int slots) { s = (int)(it % (uint32_t)slots); ph = (it / (uint32_t)slots) & 1u; }
    __device__ __forceinline__ void next(int slots) { if (++s == slots) { s = 0; ph ^= 1u; } }
};

// balanced contiguous split of n chunks over `parts` CTAs
__device__ __forceinline__ void split_range(int n, int parts, int idx, int &begin, int &end)
{
    const int base = n / parts, rem = n % parts;
    begin = idx * base + (idx < rem ? idx : rem);
    end = begin + base + (idx < rem ? 1 : 0);
}

// ------------------------------------------------------------------------------------ the kernel

// L: envelopes per adapter (scale triples over the same carriers), 1 or 2 (= B.ell).
template <int L>
__global__ void __launch_bounds__(kThreads, 1)
tc_forward_kernel(const __grid_constant__ TcBatch B)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *sm = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const uint32_t sm_base = smem_u32(sm);

    const int r = B.r, kp = B.kp, S = B.slots, C = B.cluster;
    const int RT = L * r;                  // columns of u over all envelopes
    const int tile_rows = B.tile_rows;
    // Programmatic dependent launch, same protocol as the streaming kernel.  A launch that must
    // see what ran before it sets up, waits for it, and only then lets its successor in.  A launch
    // that is independent of its predecessor (a later group of projections of the same batched
    // call) lets its successor in at once, works without waiting, and waits just before it exits,
    // so that "this grid is complete" still implies "everything before it is complete".  With
    // one CTA per SM the successor's CTAs start as this grid's CTAs leave: no idle tail between
    // the launches of one call.
    if (!B.wait_prev) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const SmemPlan plan = make_plan(r, kp, S, tile_rows, C, L);
    const uint32_t box_bytes = (uint32_t)tile_rows * kChunk * 2;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t crank = cluster_ctarank();
    const int cid = (int)cluster_id_x(), n_clusters = (int)n_cluster_id_x();

    // barriers
    const uint32_t bar0 = sm_base + plan.off_bar;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };             // x / y box landed + operand generated
    auto bar_empty = [&](int s) { return bar0 + 8u * (S + s); };      // slot may be refilled
    auto bar_raw = [&](int s) { return bar0 + 8u * (2 * S + s); };    // raw scales + sign bytes landed
    const uint32_t bar_u_full = bar0 + 8u * (3 * S);
    const uint32_t bar_z_full = bar0 + 8u * (3 * S + 1);
    const uint32_t bar_rx_full = bar0 + 8u * (3 * S + 2);
    auto bar_v_full = [&](int b) { return bar0 + 8u * (3 * S + 3 + b); };
    auto bar_v_empty = [&](int b) { return bar0 + 8u * (3 * S + 5 + b); };
    auto bar_op_full = [&](int o) { return bar0 + 8u * (3 * S + 8 + o); };           // operand tile generated
    auto bar_op_empty = [&](int o) { return bar0 + 8u * (3 * S + 8 + kOps + o); };   // MMAs that read it are done
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sm + plan.off_misc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + plan.off_misc + 4);
    const WaitCtx wctx{abort_flag, B.status};

    const int kt8 = kp / 8;                 // 16-byte chunks per row of a stage-2 operand
    const int r8 = r / 8;
    const int rt8 = RT / 8;
    const bool half_io = B.io != kIoBf16;       // x, y and W1 are IEEE halves
    const bool lo_pass = B.io != kIoF16Exact;   // W1 and U carry low parts of s_in
    const uint32_t sign_bytes = 8u * r;     // sign bytes next to one 64-column chunk, either stage
    const uint32_t raw_bytes = 256u * L + sign_bytes;   // + one 64-entry scale row per envelope

    // ---- one-time setup ---------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(bar_full(s), 1);                 // the producer's expect_tx arrive
            mbar_init(bar_empty(s), 1);
            mbar_init(bar_raw(s), 1);
        }
        for (int o = 0; o < kOps; ++o) {
            mbar_init(bar_op_full(o), kGenGroupThreads);
            mbar_init(bar_op_empty(o), 1);
        }
        mbar_init(bar_u_full, 1);
        mbar_init(bar_z_full, (uint32_t)(tile_rows * rt8));  // one arrive per (row, 8-wide piece), all owners
        mbar_init(bar_rx_full, (uint32_t)(2 * tile_rows));   // one arrive per (token row, column half)
        mbar_init(bar_v_full(0), 1);
        mbar_init(bar_v_full(1), 1);
        mbar_init(bar_v_empty(0), kEpiThreads / 2);      // the epilogue group that reads the buffer
        mbar_init(bar_v_empty(1), kEpiThreads / 2);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols(L)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // stage-2 A operands start as zeros (K padding beyond r and rows beyond tile_rows stay zero)
    for (int i = tid; i < 2 * L * plan.z_bytes / 16; i += kThreads)
        reinterpret_cast<uint4 *>(sm + plan.off_z)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    cluster_sync_all();
    const uint32_t tmem_base = *tmem_slot;
    if (B.wait_prev) {
        // nothing before this line touched global memory
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }

    const int rows_per = tile_rows / C;      // token rows of a tile owned by each CTA of the cluster

    // Every role walks the same sequence of (tile, chunk) and derives slot and phase from `it`.
    uint32_t it = 0;        // chunk counter (ring position)
    uint32_t vit = 0;       // stage-2 chunk counter (TMEM accumulator double buffer)
    uint32_t tile_n = 0;    // tiles done by this cluster (phase of the per-tile barriers)

    // The launch's tiles are in order of falling cost and go to the clusters round-robin, wave by
    // wave: after the full waves cluster 0 carries the most and the last cluster the least, so
    // the last wave (the cheapest tiles, often a partial wave) is dealt from the other end.  Only
    // for three to five waves: with two the ends carry the same, and with many (the launches of a
    // full model's call, which also hand their SMs to the next launch as they finish) it measured
    // 1 - 2 % behind.
    const int last_wave = (B.total_tiles - 1) / n_clusters;
    const bool deal_back = last_wave > 1 && last_wave <= 4;
    for (int wave = 0; wave <= last_wave; ++wave, ++tile_n) {
        const int item = wave * n_clusters + ((wave == last_wave && deal_back) ? n_clusters - 1 - cid : cid);
        if (item >= B.total_tiles) break;
        // the projection of this tile: the last one whose first tile is not beyond it (a binary
        // search, seven uniform constant loads; a linear walk through the large parameter block was
        // measured at 6 % of a tile's time)
        int pi = 0;
        for (int step = 64; step > 0; step >>= 1)
            if (pi + step < B.n_proj && B.p[pi + step].tile_start <= item) pi += step;
        const TcProj &P = B.p[pi];
        const int t0 = (item - P.tile_start) * tile_rows;
        int kb, ke, nb, ne;
        split_range(P.nk, C, (int)crank, kb, ke);
        split_range(P.nn, C, (int)crank, nb, ne);
        const uint32_t tphase = tile_n & 1u;

        if (warp == 0) {
            // ================= TMA producer =================
            // Per chunk: the raw scale values (256 B) and sign bytes (8r B) that belong to the
            // chunk's 64 columns, then the 64-column box of x (stage 1) or y (stage 2).  A ragged
            // last chunk (fewer than 64 valid columns) leaves the raw fetch to the generators.
            if (lane == 0) {
                RingPos rp;
                rp.set(it, S);
                for (int c = kb; c < ke; ++c, ++it, rp.next(S)) {
                    const int s = rp.s; const uint32_t ph = rp.ph;
                    // once a wait has given up nothing more is requested: no copy may be in flight
                    // when the CTA leaves
                    if (!mbar_wait<false>(wctx, bar_empty(s), ph ^ 1u, kDevTmaWaitTimeout)) continue;
                    if ((int)it == B.skip_item) continue;      // test-hooks build only
                    const uint32_t slot = sm_base + s * plan.slot_stride;
                    const uint32_t rawdst = slot + plan.slot_data;
                    if ((c + 1) * kChunk <= P.d_in) {
                        mbar_arrive_expect_tx(bar_raw(s), raw_bytes);
#pragma unroll
                        for (int e = 0; e < L; ++e)
                            bulk_load(rawdst + 256u * e, P.s_in + (size_t)e * P.d_in + (size_t)c * kChunk, 256u, bar_raw(s));
                        bulk_load(rawdst + plan.raw_sign, reinterpret_cast<const uint8_t *>(P.packed_A) + (size_t)c * sign_bytes,
                                  sign_bytes, bar_raw(s));
                    } else {
                        mbar_arrive(bar_raw(s));
                    }
                    mbar_arrive_expect_tx(bar_full(s), box_bytes);
                    tma_load_2d(slot, &P.x_map, c * kChunk, t0, bar_full(s));
                }
                for (int c = nb; c < ne; ++c, ++it, rp.next(S)) {
                    const int s = rp.s; const uint32_t ph = rp.ph;
                    if (!mbar_wait<false>(wctx, bar_empty(s), ph ^ 1u, kDevTmaWaitTimeout)) continue;
                    if ((int)it == B.skip_item) continue;      // test-hooks build only
                    const uint32_t slot = sm_base + s * plan.slot_stride;
                    const uint32_t rawdst = slot + plan.slot_data;
                    if ((c + 1) * kChunk <= P.d_out) {
                        mbar_arrive_expect_tx(bar_raw(s), raw_bytes);
#pragma unroll
                        for (int e = 0; e < L; ++e)
                            bulk_load(rawdst + 256u * e, P.s_out + (size_t)e * P.d_out + (size_t)c * kChunk, 256u, bar_raw(s));
                        bulk_load(rawdst + plan.raw_sign, reinterpret_cast<const uint8_t *>(P.packed_B) + (size_t)c * sign_bytes,
                                  sign_bytes, bar_raw(s));
                    } else {
                        mbar_arrive(bar_raw(s));
                    }
                    mbar_arrive_expect_tx(bar_full(s), box_bytes);
                    tma_load_2d(slot, &P.y_map, c * kChunk, t0, bar_full(s));
                }
            }
        } else if (warp == 1) {
            // ================= MMA issuer =================
            // One thread; its per-chunk latency bounds the whole pipeline (measured: with slot and
            // phase recomputed from `it` by division and the descriptors rebuilt per MMA, a chunk
            // cost this thread ~1100 cycles in stage 1 and ~1800 in stage 2, more than the loads).
            // So: ring positions are carried, descriptor words are precomputed, loops are unrolled.
            if (lane == 0) {
                // N of stage 1: hi and lo rows, or the hi rows alone rounded up to the next legal N
                // (rows past r then hold stale operand data and feed accumulator columns nobody reads)
                const uint32_t idesc1 = instr_desc(kTileM, lo_pass ? 2 * RT : (RT + 15) / 16 * 16, half_io);
                const uint32_t idesc2 = instr_desc(kTileM, kChunk, false);      // z and W2 are always bf16
                const int ksteps2 = kp / 16;
                // descriptor words (layout above): low = address >> 4 | (lbo >> 4) << 16,
                // high = sbo >> 4 | version | layout << 29
                // (a shared address carries the CTA's rank in the cluster above bit 18: masked off)
                const uint32_t base18 = sm_base & 0x3ffffu;
                const uint32_t x_lo = (base18 >> 4) | (1u << 16), x_hi = 64u | (1u << 14) | (2u << 29);
                const uint32_t op_lo = ((base18 + plan.off_ops) >> 4) | (8u << 16);
                const uint32_t w1_hi = 64u | (1u << 14);
                const uint32_t z_hi = (uint32_t)(kt8 * 8) | (1u << 14);
                const uint32_t zhi_lo = ((base18 + plan.off_z) >> 4) | (8u << 16);          // envelope 0, hi tile
                const uint32_t z_units = (uint32_t)plan.z_bytes >> 4;                       // hi -> lo, lo -> next envelope
                const uint32_t slot_units = (uint32_t)plan.slot_stride >> 4, op_units = (uint32_t)plan.op_bytes >> 4;
                uint32_t s = it % S, ph = (it / S) & 1u, o = it % kOps, oph = (it / kOps) & 1u;
                for (int c = kb; c < ke; ++c, ++it) {
                    // after a wait that gave up no MMA is issued any more (the commits below still
                    // arrive, so every role keeps walking its chunks and reaches the teardown)
                    bool ok = mbar_wait<false>(wctx, bar_full(s), ph, kDevMmaWaitTimeout);
                    ok = mbar_wait<false>(wctx, bar_op_full(o), oph, kDevMmaWaitTimeout) && ok;
                    tc_fence_after();
                    const uint32_t a_lo = x_lo + s * slot_units;          // x tile, 128B swizzle
                    const uint32_t b_lo = op_lo + o * op_units;           // W1, no swizzle
                    if (ok) {
#pragma unroll
                        for (int ks = 0; ks < kChunk / 16; ++ks)
                            mma_bf16_words(tmem_base + kTmemU, a_lo + 2u * ks, x_hi, b_lo + 16u * ks, w1_hi, idesc1,
                                           (c > kb || ks > 0) ? 1u : 0u);
                    }
                    mma_commit(bar_empty(s));
                    mma_commit(bar_op_empty(o));
                    if (++s == (uint32_t)S) { s = 0; ph ^= 1u; }
                    if (++o == (uint32_t)kOps) { o = 0; oph ^= 1u; }
                }
                mma_commit(bar_u_full);
                mbar_wait<true>(wctx, bar_z_full, tphase, kDevMmaWaitTimeout);
                fence_proxy_async();
                tc_fence_after();
                uint32_t vb = vit & 1u, vph = (vit >> 1) & 1u;
                for (int c = nb; c < ne; ++c, ++it, ++vit) {
                    bool ok = mbar_wait<false>(wctx, bar_op_full(o), oph, kDevMmaWaitTimeout);   // the y box is not needed here
                    ok = mbar_wait<false>(wctx, bar_v_empty(vb), vph ^ 1u, kDevMmaWaitTimeout) && ok;
                    tc_fence_after();
                    const uint32_t b_lo = op_lo + o * op_units;           // W2, no swizzle
                    // one accumulator per envelope: V_e = Z_e,hi W2^T + Z_e,lo W2^T over the same W2
                    if (ok) {
#pragma unroll
                        for (int e = 0; e < L; ++e) {
                            const uint32_t d = tmem_base + kTmemV + (vb * L + e) * kChunk;
                            const uint32_t zh_lo = zhi_lo + 2u * e * z_units, zl_lo = zh_lo + z_units;
#pragma unroll
                            for (int ks = 0; ks < kMaxRank / 16; ++ks)
                                if (ks < ksteps2)
                                    mma_bf16_words(d, zh_lo + 16u * ks, z_hi, b_lo + 16u * ks, z_hi, idesc2, ks > 0 ? 1u : 0u);
#pragma unroll
                            for (int ks = 0; ks < kMaxRank / 16; ++ks)
                                if (ks < ksteps2)
                                    mma_bf16_words(d, zl_lo + 16u * ks, z_hi, b_lo + 16u * ks, z_hi, idesc2, 1u);
                        }
                    }
                    mma_commit(bar_v_full(vb));
                    mma_commit(bar_op_empty(o));
                    if (++o == (uint32_t)kOps) { o = 0; oph ^= 1u; }
                    vph ^= vb;              // the phase flips when the buffer index wraps from 1 to 0
                    vb ^= 1u;
                }
            }
        } else if (warp < 2 + kGenThreads / 32) {
            // ================= operand generators =================
            const int group = (tid - 64) / kGenGroupThreads;    // this thread's generator group
            const int g = (tid - 64) % kGenGroupThreads;        // 0..kGenGroupThreads-1 within the group
            const int rsub = g & 7;                // row within an 8-row core matrix
            const int cc = (g >> 3) & 7;           // 16-byte chunk (8 columns) within the 64-column box
            const int kg0 = g >> 6;                // first 8-row group handled by this thread (stage 1)
            RingPos rp;
            rp.set(it, S);
            for (int c = kb; c < ke; ++c, ++it, rp.next(S)) {
                if ((int)(it % kGenGroups) != group) continue;
                const int s = rp.s; const uint32_t ph = rp.ph;
                mbar_wait<false>(wctx, bar_raw(s), ph, kDevTmaWaitTimeout);
                const int o = it % kOps;
                mbar_wait<false>(wctx, bar_op_empty(o), ((it / kOps) & 1u) ^ 1u, kDevMmaWaitTimeout);
                uint8_t *aux = sm + plan.off_ops + o * plan.op_bytes;
                float *raw_scale = reinterpret_cast<float *>(sm + s * plan.slot_stride + plan.slot_data);
                uint8_t *raw_sign = reinterpret_cast<uint8_t *>(raw_scale) + plan.raw_sign;
                if ((c + 1) * kChunk > P.d_in) {
                    // ragged last chunk: guarded loads (the sign block itself is always complete)
                    for (int idx = g; idx < L * kChunk; idx += kGenGroupThreads) {
                        const int e = idx >> 6, col = c * kChunk + (idx & 63);
                        raw_scale[idx] = (col < P.d_in) ? __ldg(P.s_in + (size_t)e * P.d_in + col) : 0.0f;
                    }
                    for (int w = g; w < 2 * r; w += kGenGroupThreads)
                        reinterpret_cast<uint32_t *>(raw_sign)[w] = __ldg(P.packed_A + (size_t)c * 2 * r + w);
                    asm volatile("bar.sync %0, %1;" ::"r"(2 + group), "n"(kGenGroupThreads) : "memory");
                }
                // s_in of this thread's 8 columns (every envelope's), split into bf16 hi + bf16 lo
                uint32_t hi[L][4], lo[L][4];
#pragma unroll
                for (int e = 0; e < L; ++e) {
                    const float4 sa = *reinterpret_cast<const float4 *>(raw_scale + e * kChunk + cc * 8);
                    const float4 sb = *reinterpret_cast<const float4 *>(raw_scale + e * kChunk + cc * 8 + 4);
                    const float sv[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        if (half_io) {
                            hi[e][p] = pack2_f16(sv[2 * p], sv[2 * p + 1]);
                            const float2 hf = unpack2_f16(hi[e][p]);
                            lo[e][p] = pack2_f16(sv[2 * p] - hf.x, sv[2 * p + 1] - hf.y);
                        } else {
                            const float ah = bf16_round(sv[2 * p]), bh = bf16_round(sv[2 * p + 1]);
                            hi[e][p] = pack2_bf16(ah, bh);
                            lo[e][p] = pack2_bf16(sv[2 * p] - ah, sv[2 * p + 1] - bh);
                        }
                    }
                }
                // W1 rows: envelope e, rank k -> hi row e r + k, lo row ell r + e r + k (the same signs
                // under every envelope's scales)
                uint8_t *w1 = aux;
                for (int k = kg0 * 8 + rsub; k < r; k += kGenGroupThreads / 8) {
                    const uint4 m = sign_masks(raw_sign[k * 8 + cc]);
#pragma unroll
                    for (int e = 0; e < L; ++e) {
                        const int row_hi = e * r + k, row_lo = RT + row_hi;
                        *reinterpret_cast<uint4 *>(w1 + (row_hi >> 3) * 1024 + cc * 128 + (row_hi & 7) * 16) =
                            make_uint4(hi[e][0] ^ m.x, hi[e][1] ^ m.y, hi[e][2] ^ m.z, hi[e][3] ^ m.w);
                        if (lo_pass)
                            *reinterpret_cast<uint4 *>(w1 + (row_lo >> 3) * 1024 + cc * 128 + (row_lo & 7) * 16) =
                                make_uint4(lo[e][0] ^ m.x, lo[e][1] ^ m.y, lo[e][2] ^ m.z, lo[e][3] ^ m.w);
                    }
                }
                fence_proxy_async();
                mbar_arrive(bar_op_full(o));
            }
            for (int c = nb; c < ne; ++c, ++it, rp.next(S)) {
                if ((int)(it % kGenGroups) != group) continue;
                const int s = rp.s; const uint32_t ph = rp.ph;
                mbar_wait<false>(wctx, bar_raw(s), ph, kDevTmaWaitTimeout);
                const int o = it % kOps;
                mbar_wait<false>(wctx, bar_op_empty(o), ((it / kOps) & 1u) ^ 1u, kDevMmaWaitTimeout);
                uint8_t *aux = sm + plan.off_ops + o * plan.op_bytes;
                float *raw_scale = reinterpret_cast<float *>(sm + s * plan.slot_stride + plan.slot_data);
                uint8_t *raw_sign = reinterpret_cast<uint8_t *>(raw_scale) + plan.raw_sign;
                if ((c + 1) * kChunk > P.d_out) {
                    const int64_t n_words = ((int64_t)P.d_out * r + 31) / 32;
                    for (int idx = g; idx < L * kChunk; idx += kGenGroupThreads) {
                        const int e = idx >> 6, col = c * kChunk + (idx & 63);
                        raw_scale[idx] = (col < P.d_out) ? __ldg(P.s_out + (size_t)e * P.d_out + col) : 0.0f;
                    }
                    for (int w = g; w < 2 * r; w += kGenGroupThreads) {
                        const int64_t gw = (int64_t)c * 2 * r + w;
                        reinterpret_cast<uint32_t *>(raw_sign)[w] = (gw < n_words) ? __ldg(P.packed_B + gw) : 0u;
                    }
                    asm volatile("bar.sync %0, %1;" ::"r"(2 + group), "n"(kGenGroupThreads) : "memory");
                }
                uint8_t *w2 = aux;
                // 64 rows x kt8 chunks; task = (row group, chunk, row in group)
                for (int task = g; task < kChunk * kt8; task += kGenGroupThreads) {
                    const int rs = task & 7;
                    const int ch = (task >> 3) % kt8;
                    const int row = ((task >> 3) / kt8) * 8 + rs;
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (c * kChunk + row < P.d_out && ch < r8) {
                        const uint4 m = sign_masks(raw_sign[row * r8 + ch]);
                        v = make_uint4(0x3f803f80u ^ m.x, 0x3f803f80u ^ m.y, 0x3f803f80u ^ m.z, 0x3f803f80u ^ m.w);
                    }
                    *reinterpret_cast<uint4 *>(w2 + (row >> 3) * (kt8 * 128) + ch * 128 + rs * 16) = v;
                }
                fence_proxy_async();
                mbar_arrive(bar_op_full(o));
            }
        } else {
            // ================= epilogue (8 warps: 4 TMEM lane quadrants x 2 column halves) ==========
            const int e = tid - (64 + kGenThreads);       // 0..kEpiThreads-1
            const int quad = warp & 3;                    // TMEM lanes 32*quad .. 32*quad+31
            const int chalf = e >> 7;                     // which 32 of a chunk's 64 columns
            const int row = quad * 32 + lane;             // token row of the tile
            const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16);
            const bool warp_has_rows = quad * 32 < tile_rows;    // warp-uniform
            const bool row_valid = row < tile_rows;
            it += (ke - kb);

            // ---- after stage 1: partial u -> owner CTA of this row (even pieces: half 0, odd: half 1)
            mbar_wait<false>(wctx, bar_u_full, tphase, kDevEpilogueWaitTimeout);
            __syncwarp();
            tc_fence_after();
            if (C == 1) {
                // no exchange: this thread's pieces of u go straight to z = s_r * u as bf16 hi + lo
                if (warp_has_rows) {
                    // piece p = columns 8p .. 8p+7 of u = envelope p / r8, ranks 8 (p % r8) ..; s_r is
                    // ell x r row-major, so its flat index is the column of u
                    for (int p = chalf; p < rt8; p += 2) {
                        float h[8], l[8];
                        tmem_ld8(tlane + kTmemU + p * 8, h);          // warp-collective
                        if (lo_pass) {
                            tmem_ld8(tlane + kTmemU + RT + p * 8, l);
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) l[i] = 0.0f;
                        }
                        tmem_wait_ld();
                        if (row_valid) {
                            uint32_t zh[4], zl[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float z0 = (h[2 * q] + l[2 * q]) * __ldg(P.s_r + p * 8 + 2 * q);
                                const float z1 = (h[2 * q + 1] + l[2 * q + 1]) * __ldg(P.s_r + p * 8 + 2 * q + 1);
                                const float h0 = bf16_round(z0), h1 = bf16_round(z1);
                                zh[q] = pack2_bf16(h0, h1);
                                zl[q] = pack2_bf16(z0 - h0, z1 - h1);
                            }
                            const int env = (L == 1) ? 0 : p / r8, pe = p - env * r8;
                            const uint32_t off = (uint32_t)(env * 2 * plan.z_bytes + (row >> 3) * (kt8 * 128) + pe * 128 + (row & 7) * 16);
                            *reinterpret_cast<uint4 *>(sm + plan.off_z + off) = make_uint4(zh[0], zh[1], zh[2], zh[3]);
                            *reinterpret_cast<uint4 *>(sm + plan.off_z + plan.z_bytes + off) = make_uint4(zl[0], zl[1], zl[2], zl[3]);
                            fence_proxy_async();
                            mbar_arrive(bar_z_full);
                        }
                    }
                    tc_fence_before();
                }
            } else {
            if (warp_has_rows) {
                const uint32_t owner = row_valid ? (uint32_t)(row / rows_per) : 0u;
                const int row_local = row - (int)owner * rows_per;
                const uint32_t rx_remote = mapa(sm_base + plan.off_rx, owner) +
                                           (uint32_t)(((int)crank * rows_per + row_local) * RT) * 4u;
                for (int p = chalf; p < rt8; p += 2) {
                    float h[8], l[8];
                    tmem_ld8(tlane + kTmemU + p * 8, h);          // warp-collective
                    if (lo_pass) {
                        tmem_ld8(tlane + kTmemU + RT + p * 8, l);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) l[i] = 0.0f;
                    }
                    tmem_wait_ld();
                    if (row_valid) {
                        uint32_t w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) w[i] = __float_as_uint(h[i] + l[i]);
                        st_cluster_v4(rx_remote + p * 32, w[0], w[1], w[2], w[3]);
                        st_cluster_v4(rx_remote + p * 32 + 16, w[4], w[5], w[6], w[7]);
                    }
                }
                tc_fence_before();
                if (row_valid) mbar_arrive_remote(mapa(bar_rx_full, owner));
            }
            // ---- owner: reduce over source CTAs in a fixed order, scale by s_r, split, broadcast z
            mbar_wait<true>(wctx, bar_rx_full, tphase, kDevClusterWaitTimeout);
            {
                const float *rx = reinterpret_cast<const float *>(sm + plan.off_rx);
                for (int task = e; task < rows_per * rt8; task += kEpiThreads) {
                    const int row_local = task / rt8, p = task - row_local * rt8;
                    float u[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) u[i] = 0.0f;
                    for (int src = 0; src < C; ++src) {
                        const float4 a = *reinterpret_cast<const float4 *>(rx + (src * rows_per + row_local) * RT + p * 8);
                        const float4 b = *reinterpret_cast<const float4 *>(rx + (src * rows_per + row_local) * RT + p * 8 + 4);
                        u[0] += a.x; u[1] += a.y; u[2] += a.z; u[3] += a.w;
                        u[4] += b.x; u[5] += b.y; u[6] += b.z; u[7] += b.w;
                    }
                    uint32_t zh[4], zl[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float z0 = u[2 * q] * __ldg(P.s_r + p * 8 + 2 * q);
                        const float z1 = u[2 * q + 1] * __ldg(P.s_r + p * 8 + 2 * q + 1);
                        const float h0 = bf16_round(z0), h1 = bf16_round(z1);
                        zh[q] = pack2_bf16(h0, h1);
                        zl[q] = pack2_bf16(z0 - h0, z1 - h1);
                    }
                    const int grow = (int)crank * rows_per + row_local;          // row within the tile
                    const int env = (L == 1) ? 0 : p / r8, pe = p - env * r8;
                    const uint32_t off = (uint32_t)(env * 2 * plan.z_bytes + (grow >> 3) * (kt8 * 128) + pe * 128 + (grow & 7) * 16);
                    for (int dst = 0; dst < C; ++dst) {
                        const uint32_t zb = mapa(sm_base + plan.off_z, dst) + off;
                        st_cluster_v4(zb, zh[0], zh[1], zh[2], zh[3]);
                        st_cluster_v4(zb + plan.z_bytes, zl[0], zl[1], zl[2], zl[3]);
                    }
                    asm volatile("fence.proxy.async.shared::cluster;" ::: "memory");
                    for (int dst = 0; dst < C; ++dst) mbar_arrive_remote(mapa(bar_z_full, dst));
                }
            }
            }
            // ---- after stage 2: y tile (already in the slot) += s_out * V, in place, then TMA store.
            // The two groups of four warps (one TMEM lane quadrant each) take alternate chunks, so
            // that one group's TMEM load, barrier and store latencies overlap the other's
            // arithmetic; chunk parity is also the accumulator buffer, so group g always reads
            // buffer g.  A thread handles all 64 columns of its token row.
            const int egroup = chalf;
            const bool store_thread = (e & (kEpiThreads / 2 - 1)) == 0;
            int prev_slot = -1;
            RingPos rp;
            rp.set(it, S);
            for (int c = nb; c < ne; ++c, ++it, ++vit, rp.next(S)) {
                if ((int)(vit & 1u) != egroup) continue;
                const int s = rp.s; const uint32_t ph = rp.ph;
                const int vb = egroup; const uint32_t vph = (vit >> 1) & 1u;
                mbar_wait<false>(wctx, bar_v_full(vb), vph, kDevEpilogueWaitTimeout);
                mbar_wait<false>(wctx, bar_full(s), ph, kDevEpilogueWaitTimeout);
                __syncwarp();
                tc_fence_after();
                uint8_t *ytile = sm + s * plan.slot_stride;
                const float *so = reinterpret_cast<const float *>(ytile + plan.slot_data);
                if (warp_has_rows && L == 2) {
                    // two envelopes: y += s_out[0] * V_0 + s_out[1] * V_1, 16 columns at a time
#pragma unroll
                    for (int qq = 0; qq < 4; ++qq) {
                        uint32_t v0[16], v1[16];
                        tmem_ld16(tlane + kTmemV + (2 * vb) * kChunk + qq * 16, v0);       // warp-collective
                        tmem_ld16(tlane + kTmemV + (2 * vb + 1) * kChunk + qq * 16, v1);
                        tmem_wait_ld();
                        if (qq == 3) {
                            tc_fence_before();
                            mbar_arrive(bar_v_empty(vb));
                        }
                        if (row_valid) {
#pragma unroll
                            for (int q = 0; q < 2; ++q) {
                                const int ch = qq * 2 + q;                     // 16-byte chunk of the row
                                uint4 *py = reinterpret_cast<uint4 *>(ytile + row * 128 + ((ch ^ (row & 7)) * 16));
                                const uint4 yv = *py;
                                const float4 s0 = *reinterpret_cast<const float4 *>(so + ch * 8);
                                const float4 s1 = *reinterpret_cast<const float4 *>(so + ch * 8 + 4);
                                const float4 t0 = *reinterpret_cast<const float4 *>(so + kChunk + ch * 8);
                                const float4 t1 = *reinterpret_cast<const float4 *>(so + kChunk + ch * 8 + 4);
                                const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w};
                                const float sc0[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
                                const float sc1[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
                                uint32_t ow[4];
#pragma unroll
                                for (int k2 = 0; k2 < 4; ++k2) {
                                    float y0, y1;
                                    if (half_io) {
                                        const float2 yf = unpack2_f16(yw[k2]);
                                        y0 = yf.x; y1 = yf.y;
                                    } else {
                                        y0 = __uint_as_float(yw[k2] << 16);
                                        y1 = __uint_as_float(yw[k2] & 0xffff0000u);
                                    }
                                    float o0 = fmaf(sc0[2 * k2], __uint_as_float(v0[q * 8 + 2 * k2]), y0);
                                    float o1 = fmaf(sc0[2 * k2 + 1], __uint_as_float(v0[q * 8 + 2 * k2 + 1]), y1);
                                    o0 = fmaf(sc1[2 * k2], __uint_as_float(v1[q * 8 + 2 * k2]), o0);
                                    o1 = fmaf(sc1[2 * k2 + 1], __uint_as_float(v1[q * 8 + 2 * k2 + 1]), o1);
                                    ow[k2] = half_io ? pack2_f16(o0, o1) : pack2_bf16(o0, o1);
                                }
                                *py = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                            }
                        }
                    }
                } else if (warp_has_rows) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        uint32_t v[32];
                        tmem_ld32(tlane + kTmemV + vb * kChunk + hh * 32, v);   // warp-collective
                        tmem_wait_ld();
                        if (hh == 1) {
                            tc_fence_before();
                            mbar_arrive(bar_v_empty(vb));
                        }
                        if (row_valid) {
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int ch = hh * 4 + q;                     // 16-byte chunk of the row
                                uint4 *py = reinterpret_cast<uint4 *>(ytile + row * 128 + ((ch ^ (row & 7)) * 16));
                                const uint4 yv = *py;
                                const float4 s0 = *reinterpret_cast<const float4 *>(so + ch * 8);
                                const float4 s1 = *reinterpret_cast<const float4 *>(so + ch * 8 + 4);
                                const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w};
                                const float sc[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
                                uint32_t ow[4];
#pragma unroll
                                for (int k2 = 0; k2 < 4; ++k2) {
                                    float y0, y1;
                                    if (half_io) {
                                        const float2 yf = unpack2_f16(yw[k2]);
                                        y0 = yf.x; y1 = yf.y;
                                    } else {
                                        y0 = __uint_as_float(yw[k2] << 16);
                                        y1 = __uint_as_float(yw[k2] & 0xffff0000u);
                                    }
                                    const float o0 = fmaf(sc[2 * k2], __uint_as_float(v[q * 8 + 2 * k2]), y0);
                                    const float o1 = fmaf(sc[2 * k2 + 1], __uint_as_float(v[q * 8 + 2 * k2 + 1]), y1);
                                    ow[k2] = half_io ? pack2_f16(o0, o1) : pack2_bf16(o0, o1);
                                }
                                *py = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                            }
                        }
                    }
                } else {
                    mbar_arrive(bar_v_empty(vb));
                }
                fence_proxy_async();
                asm volatile("bar.sync %0, %1;" ::"r"(1 + 3 * egroup), "n"(kEpiThreads / 2) : "memory");
                if (store_thread) {
                    // a CTA in which any wait gave up writes nothing more: what sits in the slot may be
                    // built on incomplete sums (the flag was raised before anything that depends on the
                    // missing data could reach this point)
                    if (!*abort_flag) tma_store_2d(&P.y_map, sm_base + s * plan.slot_stride, c * kChunk, t0);
                    bulk_commit();
                    if (prev_slot >= 0) {
                        bulk_wait_read_1();
                        mbar_arrive(bar_empty(prev_slot));
                    }
                    prev_slot = s;
                }
            }
            if (store_thread && prev_slot >= 0) {
                bulk_wait_read_0();
                mbar_arrive(bar_empty(prev_slot));
            }
        }
    }

    // ---- teardown -------------------------------------------------------------------------------
    if (tid == 64 + kGenThreads || tid == 64 + kGenThreads + kEpiThreads / 2) bulk_wait_all();   // the threads that issued the stores
    if (*abort_flag) {
        // give copies that may still be in flight time to land before the CTA goes away
        const long long start = clock64();
        while (clock64() - start < 2000000LL) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols(L)) : "memory");
    }
    if (!B.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");
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

// T x d bf16 matrix with row pitch ld (elements); boxes of 128 rows x 64 columns, 128B swizzle.
bool make_map(CUtensorMap *map, const void *base, int64_t T, int64_t d, int64_t ld, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)T};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kChunk, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

struct LaunchShape { int cluster, tile_rows, slots, smem, max_clusters; };

constexpr int kMaxSlots = 32;

const void *kernel_for(int ell)
{
    return ell == 2 ? reinterpret_cast<const void *>(&tc_forward_kernel<2>)
                    : reinterpret_cast<const void *>(&tc_forward_kernel<1>);
}

// Co-resident clusters for an instantiation, a cluster size and a shared-memory footprint (cached:
// the query is slow).
int max_active_clusters(int ell, int cluster, int smem)
{
    static std::mutex mu;
    static int cache_ell[64], cache_cluster[64], cache_smem[64], cache_val[64], n_cached = 0;
    static bool attr_set = false;
    std::lock_guard<std::mutex> lock(mu);
    if (!attr_set) {
        for (int l = 1; l <= kMaxTcEll; ++l)
            if (cudaFuncSetAttribute(kernel_for(l), cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) !=
                cudaSuccess) {
                cudaGetLastError();
                return 0;
            }
        attr_set = true;
    }
    for (int i = 0; i < n_cached; ++i)
        if (cache_ell[i] == ell && cache_cluster[i] == cluster && cache_smem[i] == smem) return cache_val[i];
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(cluster, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = cluster; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel_for(ell), &cfg) != cudaSuccess) {
        cudaGetLastError();
        n = 0;
    }
    if (n_cached < 64) {
        cache_ell[n_cached] = ell;
        cache_cluster[n_cached] = cluster; cache_smem[n_cached] = smem; cache_val[n_cached] = n;
        ++n_cached;
    }
    return n;
}

// Deepest ring that fits next to the fixed buffers, and how many clusters can be co-resident.
bool plan_launch(int r, int kp, int ell, int cluster, int tile_rows, LaunchShape *out)
{
    int slots = 0;
    for (int s = kMaxSlots; s >= 2; --s) {
        if (make_plan(r, kp, s, tile_rows, cluster, ell).total + 1024 <= kSmemBudget) { slots = s; break; }
    }
    if (slots < 2) return false;
    const int smem = make_plan(r, kp, slots, tile_rows, cluster, ell).total + 1024;
    const int n = max_active_clusters(ell, cluster, smem);
    if (n < 1) return false;
    out->cluster = cluster; out->tile_rows = tile_rows; out->slots = slots; out->smem = smem;
    out->max_clusters = n;
    return true;
}

// Choose cluster size and tile height for a launch whose projections hold `tokens` token rows in
// all (tiles_for(rows) = tiles of the launch at a given tile height).  Few tokens are spread over many SMs by splitting
// the feature axes over a cluster and by shortening the tile; many tokens use tall tiles and small
// clusters.
template <typename TilesFor>
bool choose_shape(int r, int kp, int ell, int64_t tokens, int64_t full_tiles, int min_chunks, TilesFor tiles_for,
                  LaunchShape *best)
{
    double best_cost = 1e300;
    bool found = false;
    // Plenty of full-height tiles (two waves or more): no cluster, nothing to exchange.
    {
        LaunchShape solo;
        if (plan_launch(r, kp, ell, 1, kTileM, &solo) && full_tiles >= 2 * (int64_t)solo.max_clusters) {
            *best = solo;
            return true;
        }
    }
    for (int c = 8; c >= 1; c /= 2) {
        if (c > min_chunks) continue;
        LaunchShape probe;
        if (!plan_launch(r, kp, ell, c, kTileM, &probe)) continue;
        const int cap = probe.max_clusters;
        // waves of `cap` clusters needed with full-height tiles, then the tile height that fills them
        const int64_t waves = (full_tiles + cap - 1) / cap;
        int64_t rows = (tokens + cap * waves - 1) / (cap * waves);   // per-tile share
        rows = (rows + c - 1) / c * c;
        if (rows > kTileM) rows = kTileM;
        if (rows < c) rows = c;
        LaunchShape shape;
        if (!plan_launch(r, kp, ell, c, (int)rows, &shape)) continue;
        const int64_t tiles = tiles_for(rows);
        const int64_t w = (tiles + shape.max_clusters - 1) / shape.max_clusters;
        // cost model: time ~ waves * rows of work per cluster / CTAs sharing it, plus a fixed
        // per-tile cost (operand generation, MMA on padded rows, cluster exchange)
        const double per_tile = (double)rows / c + 24.0 / c + 6.0;
        const double cost = (double)w * per_tile;
        if (cost < best_cost) { best_cost = cost; *best = shape; found = true; }
    }
    return found;
}

}  // namespace

bool tc_supported(const lordba_proj &p, int64_t T, int dtype)
{
    if ((dtype != LORDBA_BF16 && dtype != LORDBA_F16) || T < 1) return false;
    // one envelope, or two whose ranks together fit the accumulator (their scale rows travel as
    // bulk copies too: every row must start on a 16-byte boundary)
    const int ell = ((p.flags >> 8) & 0xf) + 1;
    if (ell > kMaxTcEll) return false;
    if (p.r % 8 != 0 || p.r < 8 || ell * p.r > kMaxRank) return false;
    if (ell > 1 && (p.d_in % 4 || p.d_out % 4)) return false;
    if (p.d_in < kChunk || p.d_out < kChunk) return false;
    if (p.d_in > (1 << 30) || p.d_out > (1 << 30) || T > (1 << 30)) return false;
    if (reinterpret_cast<uintptr_t>(p.x) % 16 || reinterpret_cast<uintptr_t>(p.y) % 16) return false;
    if (p.ldx % 8 || p.ldy % 8) return false;
    // the raw scales and sign bytes of a chunk travel as bulk copies: 16-byte aligned sources
    if (reinterpret_cast<uintptr_t>(p.s_in) % 16 || reinterpret_cast<uintptr_t>(p.s_out) % 16 ||
        reinterpret_cast<uintptr_t>(p.packed_A) % 16 || reinterpret_cast<uintptr_t>(p.packed_B) % 16)
        return false;
    return encode_fn() != nullptr;
}

int launch_forward_tc(const lordba_proj *projs, const int64_t *tokens, int64_t T, int n, const FamilySelector &fsel,
                      LaunchSink &sink, bool batch_checked, int *launches)
{
    if (n == 0) return LORDBA_OK;
    const int dtype = fsel.dtype;
    if (dtype != LORDBA_BF16 && dtype != LORDBA_F16) return LORDBA_OK;
    int *status = nullptr;
    auto io_of = [&](const lordba_proj &q) {
        if (dtype == LORDBA_BF16) return (int)kIoBf16;
        return (q.flags & LORDBA_PROJ_SCALES_F16) ? (int)kIoF16Exact : (int)kIoF16;
    };
    int sms = 148;
    {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v >= 1)
            sms = v;
    }

    auto ell_of = [](const lordba_proj &q) { return ((q.flags >> 8) & 0xf) + 1; };
    // one launch per element / scale kind, envelope count, rank value and kMaxTcBatch projections
    int16_t all[kMaxCallProjs];
    for (int io = (dtype == LORDBA_BF16 ? kIoBf16 : kIoF16); io <= (dtype == LORDBA_BF16 ? kIoBf16 : kIoF16Exact); ++io)
    for (int ell = 1; ell <= kMaxTcEll; ++ell)
    for (int r = 8; ell * r <= kMaxRank; r += 8) {
        // all projections of this kind and rank, in order of falling cost per tile (a y chunk
        // costs about 1.7 x chunks): tiles go to the persistent CTAs round-robin in index order,
        // so a CTA's later tiles are cheaper than its earlier ones, and the last launch of the
        // call holds the cheapest projections
        int total = 0;
        int64_t total_full_tiles = 0;
        for (int i = 0; i < n; ++i) {
            const int64_t rows = rows_of(tokens, T, i);
            if (rows > 0 && projs[i].r == r && ell_of(projs[i]) == ell && io_of(projs[i]) == io &&
                fsel.family(projs[i], rows) == LORDBA_VARIANT_TC) {
                all[total++] = (int16_t)i;
                total_full_tiles += (rows + kTileM - 1) / kTileM;
            }
        }
        if (total == 0) continue;
        if (!status && !(status = device_status_word())) return LORDBA_ECUDA;
        std::sort(all, all + total, [&](int16_t a, int16_t b) {
            const int64_t ca = 10 * projs[a].d_in + 17 * projs[a].d_out, cb = 10 * projs[b].d_in + 17 * projs[b].d_out;
            return ca != cb ? ca > cb : a < b;
        });
        // Launch sizes.  The launches of a call run back to back (each one's CTAs start as the
        // previous one's leave), so only the last one's tail is exposed: it gets the number of
        // projections whose 128-token tiles fill whole waves of the SMs best, the others share
        // the rest evenly.
        int sizes[kMaxCallProjs / kMaxTcBatch + 3];
        int n_sizes = 0;
        if (total <= kMaxTcBatch) {
            sizes[n_sizes++] = total;
        } else {
            const int64_t tpp = (total_full_tiles + total - 1) / total;      // tiles per projection (mean)
            const int64_t ctas = sms;
            int last = kMaxTcBatch;
            double best_fill = 0.0;
            for (int cand = kMaxTcBatch; cand >= kMaxTcBatch / 3; --cand) {
                const int64_t tiles = cand * tpp, waves = (tiles + ctas - 1) / ctas;
                const double fill = (double)tiles / (double)(waves * ctas);
                if (fill > best_fill + 1e-9) { best_fill = fill; last = cand; }
            }
            const int rest = total - last, parts = (rest + kMaxTcBatch - 1) / kMaxTcBatch;
            for (int k = 0; k < parts; ++k) sizes[n_sizes++] = rest / parts + (k < rest % parts ? 1 : 0);
            sizes[n_sizes++] = last;
        }
        int next = 0;
        for (int li = 0; li < n_sizes; ++li) {
            const int m = sizes[li];
            const int first = next;
            next += m;
            int min_chunks = 1 << 30;
            int64_t tok_sum = 0, full_tiles = 0;
            for (int k = 0; k < m; ++k) {
                const lordba_proj &q = projs[all[first + k]];
                const int64_t rows = rows_of(tokens, T, all[first + k]);
                const int nk = (int)((q.d_in + kChunk - 1) / kChunk);
                const int nn = (int)((q.d_out + kChunk - 1) / kChunk);
                if (nk < min_chunks) min_chunks = nk;
                if (nn < min_chunks) min_chunks = nn;
                tok_sum += rows;
                full_tiles += (rows + kTileM - 1) / kTileM;
            }
            const int kp = (r + 15) / 16 * 16;
            LaunchShape shape;
            auto tiles_for = [&](int64_t tile_rows) {
                int64_t t = 0;
                for (int k = 0; k < m; ++k) t += (rows_of(tokens, T, all[first + k]) + tile_rows - 1) / tile_rows;
                return t;
            };
            if (!choose_shape(r, kp, ell, tok_sum, full_tiles, min_chunks, tiles_for, &shape)) return LORDBA_ECUDA;

            TcBatch b;
            std::memset(&b, 0, sizeof(b));
            int64_t tile_count = 0;
            for (int k = 0; k < m; ++k) {
                const lordba_proj &q = projs[all[first + k]];
                const int64_t rows = rows_of(tokens, T, all[first + k]);
                TcProj &t = b.p[k];
                if (!make_map(&t.x_map, q.x, rows, q.d_in, q.ldx, shape.tile_rows) ||
                    !make_map(&t.y_map, q.y, rows, q.d_out, q.ldy, shape.tile_rows))
                    return LORDBA_EUNSUPPORTED;
                t.packed_A = q.packed_A; t.packed_B = q.packed_B;
                t.s_in = q.s_in; t.s_r = q.s_r; t.s_out = q.s_out;
                t.d_in = (int)q.d_in; t.d_out = (int)q.d_out;
                t.nk = (int)((q.d_in + kChunk - 1) / kChunk);
                t.nn = (int)((q.d_out + kChunk - 1) / kChunk);
                t.tile_start = (int)tile_count;
                tile_count += (rows + shape.tile_rows - 1) / shape.tile_rows;
            }
            if (tile_count > (1 << 30)) return LORDBA_EUNSUPPORTED;
            b.n_proj = m;
            b.total_tiles = (int)tile_count;
            b.r = r;
            b.ell = ell;
            b.kp = kp;
            b.io = io;
            b.status = status;
            b.skip_item = test_skip_item();
            b.cluster = shape.cluster;
            b.slots = shape.slots;
            b.tile_rows = shape.tile_rows;
            // the projections of a checked batch are independent of one another: every launch
            // after the first may overlap its predecessor
            b.wait_prev = (*launches == 0 || !batch_checked) ? 1 : 0;
            ++*launches;
            const int n_clusters = b.total_tiles < shape.max_clusters ? b.total_tiles : shape.max_clusters;

            LaunchRec rec;
            std::memset(&rec, 0, sizeof(rec));
            rec.func = kernel_for(ell);
            rec.grid[0] = (unsigned)(n_clusters * shape.cluster); rec.grid[1] = 1; rec.grid[2] = 1;
            rec.block = kThreads;
            rec.smem = (uint32_t)shape.smem;
            rec.cluster = (uint32_t)shape.cluster;
            rec.pdl = 1;
            rec.n_args = 1;
            rec.arg_bytes[0] = sizeof(TcBatch);
            const int rc = sink.emit(rec, &b, nullptr);
            if (rc != LORDBA_OK) return rc;
        }
    }
    return LORDBA_OK;
}

}  // namespace lordba
