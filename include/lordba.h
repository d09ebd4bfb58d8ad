/*
 * lordba.h -- C ABI of the B200 (sm_100a) LoRDBA adapter-forward library.
 *
 * The library evaluates the unmerged low-rank double-binary adapter branch
 *
 *     y[t,:] += s_out * ( B_sign ( s_r * ( A_sign ( s_in * x[t,:] ) ) ) )      t < T
 *
 * i.e. the paper's Delta-W(theta) = D_alpha B1 D_beta B2 D_gamma (Def. 1, Eq. 4,
 * canonical l = 1) applied in the evaluation order of Eq. 8 with both binary
 * products done as the sign accumulation of Eq. 9, and added to the buffer that
 * already holds the frozen base projection's output (Eq. 2).
 *
 *     paper              here
 *     N, M, R            d_in, d_out, r
 *     B1 (N x R)         A_sign = B1^T   (r x d_in,   +-1)
 *     B2 (R x M)         B_sign = B2^T   (d_out x r,  +-1)
 *     alpha, beta, gamma s_in (d_in), s_r (r), s_out (d_out), float32
 *     X (T x N)          x, row-major, one token per row
 *
 * The paper's Def. 1 carries no scalar LoRA alpha/r factor; a caller that has
 * one multiplies it into s_r.
 *
 * Conventions for every entry point
 *   - Pointers marked [device] are caller-owned device memory of the current
 *     CUDA device; [host] pointers are ordinary host memory.  The library keeps
 *     no pointer after a call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls enqueue work on it and return without synchronising,
 *     except where stated.
 *   - Return value: a lordba_status.  Argument errors are detected on the host
 *     and nothing is launched.  There is no CPU fallback: without a usable CUDA
 *     device the calls return LORDBA_ECUDA.
 *   - Supported rank: 1 <= r <= 64.  A call takes at most LORDBA_MAX_PROJS projections
 *     (LORDBA_EUNSUPPORTED beyond that).
 *   - No entry point allocates host or device memory.
 *
 * Bit-packed carriers (the paper says only "bit-packed"; this layout is the
 * library's own).  Bit 1 <=> +1, bit 0 <=> -1, 32-bit little-endian words,
 * pad bits are 0:
 *   role 0, A carrier (r x d_in): the columns are cut into blocks of 64; block b
 *       holds r consecutive 64-bit groups, one per row k, each stored as two
 *       words (low word first).  Entry (k,i) is bit (i mod 32) of word
 *       ((i/64)*r + k)*2 + (i mod 64)/32; ceil(d_in/64)*r*2 words.  (One block is
 *       exactly what the kernels need next to one 64-column tile of x.)
 *   role 1, B carrier (d_out x r): one dense bit stream of the row-major
 *       matrix; entry (j,k) is bit (b mod 32) of word b/32 with b = j*r + k.
 */
#ifndef LORDBA_H_
#define LORDBA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LORDBA_MAX_PROJS 4096

typedef enum {
    LORDBA_F32 = 0,   /* x and y are float32                                   */
    LORDBA_BF16 = 1,  /* x and y are bfloat16; all accumulation is in float32  */
    LORDBA_F16 = 2    /* x and y are IEEE half (the precision the method exports its adapters in:
                         Sec. "Training and export", fp16 scales and activations); accumulation
                         in float32.  s_in is used as a pair of halves here: |s_in| must stay below
                         65504, and entries below 2^-14 are used with fewer than 22 bits */
} lordba_dtype;

typedef enum {
    LORDBA_OK = 0,
    LORDBA_EINVAL = 1,        /* null pointer, negative size, ld < width, x aliases y ...   */
    LORDBA_EUNSUPPORTED = 2,  /* rank outside 1..64, unknown dtype / role / variant         */
    LORDBA_EALIGN = 3,        /* a pointer is not aligned to its element type               */
    LORDBA_ECUDA = 4,         /* a CUDA runtime call or the launch failed                   */
    LORDBA_ETIMEOUT = 5,      /* a bounded device-side wait gave up (see lordba_device_status) */
    LORDBA_ETOOLARGE = 6      /* the call needs more than the library's built-in scratch buffer */
} lordba_status;

/* Kernel families the forward entry points can be pinned to (default AUTO). */
typedef enum {
    LORDBA_VARIANT_AUTO = 0,  /* the library's choice: streaming kernel where the shape allows  */
                              /* it; tcgen05 kernel for rank (x envelopes) > 16 once a call has */
                              /* enough 128-token tiles (> 32: 32 tiles, else eight per SM), and */
                              /* for widths that are not multiples of 64 from 128 tokens up     */
                              /* (rank a multiple of 8); else FMA.  lordba_query_variant tells  */
                              /* which one a given call gets                                   */
    LORDBA_VARIANT_FMA = 1,   /* CUDA-core float32 FMA kernel (always used for LORDBA_F32)  */
    LORDBA_VARIANT_TC = 2,    /* tcgen05/TMA cluster kernel; LORDBA_EUNSUPPORTED if the     */
                              /* shape or alignment rules it out                            */
    LORDBA_VARIANT_MMA = 3    /* TMA-fed streaming mma.sync kernel; LORDBA_EUNSUPPORTED if   */
                              /* the shape or alignment rules it out                        */
} lordba_variant;

/* One adapted projection for the _ex and _batched entry points.  ldx / ldy are
 * row pitches in elements (ldx >= d_in, ldy >= d_out). */
typedef struct lordba_proj {
    const void     *x;          /* [device] T x d_in,  pitch ldx                */
    const uint32_t *packed_A;   /* [device] role-0 words of A_sign (r x d_in)   */
    const uint32_t *packed_B;   /* [device] role-1 words of B_sign (d_out x r)  */
    const float    *s_in;       /* [device] d_in                                */
    const float    *s_r;        /* [device] r                                   */
    const float    *s_out;      /* [device] d_out                               */
    void           *y;          /* [device] T x d_out, pitch ldy, updated in place */
    int64_t d_in, d_out, ldx, ldy;
    int32_t r;
    int32_t flags;              /* LORDBA_PROJ_OVERLAP, _X_READY, _SCALES_F16, LORDBA_PROJ_ELL(ell); other bits 0 */
} lordba_proj;

/*
 * Multi-envelope adapters (Def. 1 / Eq. 4 with ell > 1): Delta-W is the sum of ell terms that
 * share the two sign carriers and differ in their scale triples.  A projection made with
 * LORDBA_PROJ_ELL(ell) in its flags, 1 <= ell <= LORDBA_MAX_ELL, takes s_in as ell x d_in,
 * s_r as ell x r and s_out as ell x d_out (row-major, envelope e in row e), and the call adds
 *     sum_e  s_out[e] * ( B_sign ( s_r[e] * ( A_sign ( s_in[e] * x[t,:] ) ) ) )
 * to y[t,:] with one rounding.  Flags without this field mean ell = 1.  Every envelope count at
 * every rank runs on the tensor cores (streaming kernel; two envelopes with ell * r <= 64 also
 * in the tcgen05 kernel, which the library takes for them by the same rule as for one envelope
 * of rank ell * r); the cost is about that of one envelope at rank ell * r.
 */
#define LORDBA_MAX_ELL 8
#define LORDBA_PROJ_ELL(ell) ((((ell) - 1) & 0xf) << 8)

/*
 * lordba_proj.flags: a promise by the caller that lets consecutive calls overlap on the GPU.
 * A call (all of its projections) made with LORDBA_PROJ_OVERLAP may start while the library
 * calls before it on the same stream are still running, back to and including the most recent
 * call made WITHOUT the flag.  The caller guarantees that, within such a run of calls, no call
 * reads what another one writes (a y buffer) and no call writes what another one reads or
 * writes, and that nothing else was enqueued on the stream in between.  Example: the q, k and v
 * adapters of one layer read the same x and update three different y buffers; the first is
 * called without the flag (it must see the kernel that produced x), the other two with it.
 * Work enqueued after the run is ordered after all of it, as usual.  Only the streaming
 * kernel acts on the flag; elsewhere it is accepted and ignored.
 */
#define LORDBA_PROJ_OVERLAP 1

/*
 * lordba_proj.flags: a weaker promise for a call that does depend on its predecessor, as an
 * adapter call does that follows the base projection which produced y (Eq. 2: y = W x, then
 * y += Delta-W x).  With LORDBA_PROJ_X_READY on every projection of a call made WITHOUT
 * LORDBA_PROJ_OVERLAP the caller guarantees that x, the packed carriers and the three scale
 * vectors were final before the previous piece of work on the stream began (the base projection
 * reads x itself, so this is the normal case); only y may still be in the making.  The call then
 * requests x and runs the first product (Eq. 8, u = A_sign (s_in * x)) while its predecessor
 * finishes, and touches y only once the predecessor is complete.  Only the streaming kernel acts
 * on the flag; elsewhere, and together with LORDBA_PROJ_OVERLAP, it is accepted and ignored.
 */
#define LORDBA_PROJ_X_READY 4

/*
 * lordba_proj.flags: the caller states that every entry of s_in is exactly representable as an
 * IEEE half, which is the case for an adapter exported with fp16 scales (Section 3.2: the scales
 * are trained in float32 and leave training as halves) and widened by lordba_scales_from_f16.  With
 * LORDBA_F16 activations the streaming kernel then forms x * s_in in one tensor-core pass
 * instead of two; with a false statement the low bits of s_in beyond a half are ignored, nothing
 * else.  Other kernels and dtypes accept the flag and ignore it.
 */
#define LORDBA_PROJ_SCALES_F16 2

/*
 * Widens n IEEE-half scales (the storage format of an exported adapter, 2 bytes per scale as in
 * the method's footprint count, Eq. 5) to the float32 arrays that the forward calls take.  Once
 * per adapter, like packing.  src: [device] n halves, 2-byte aligned; dst: [device] n floats.
 * Exact (every half is a float).  Asynchronous on stream.  n = 0 is a no-op; n < 0 or a null
 * pointer with n > 0 is LORDBA_EINVAL.
 */
int lordba_scales_from_f16(const uint16_t *src, float *dst, int64_t n, void *stream);

/* Number of uint32 words of a packed carrier (layout above); -1 on bad arguments. */
int64_t lordba_packed_words(int64_t rows, int64_t cols, int role);

/*
 * Bit-pack a sign matrix: the two sign carriers are kept as one bit per entry and packed
 * once per adapter (Section 3.3).  signs: [device] int8, rows x cols row-major; an entry < 0 packs
 * as -1, anything else (0 included: sign(0) = +1) as +1.  role 0: rows = r,
 * cols = d_in.  role 1: rows = d_out, cols = r.  packed: [device], at least
 * lordba_packed_words() words, fully overwritten (pad bits 0).
 */
int lordba_pack_signs(const int8_t *signs, int64_t rows, int64_t cols, int role,
                      uint32_t *packed, void *stream);

/* Inverse of lordba_pack_signs: writes +1 / -1 into signs [device] (rows x cols). */
int lordba_unpack_signs(const uint32_t *packed, int64_t rows, int64_t cols, int role,
                        int8_t *signs, void *stream);

/*
 * Adapter forward, Eq. 8 / Eq. 9, bfloat16 activations, dense rows
 * (ldx = d_in, ldy = d_out).  All pointers [device].  y is read, the adapter
 * term is added in float32 and the sum is rounded once to bfloat16.  x and y
 * must not overlap.  T = 0 is a no-op.
 */
int lordba_adapter_forward(const void *x, const uint32_t *packed_A, const uint32_t *packed_B,
                           const float *s_in, const float *s_r, const float *s_out, void *y,
                           int64_t T, int64_t d_in, int64_t d_out, int r, void *stream);

/* Same operation with float32 x and y (float32 arithmetic throughout). */
int lordba_adapter_forward_f32(const float *x, const uint32_t *packed_A, const uint32_t *packed_B,
                               const float *s_in, const float *s_r, const float *s_out, float *y,
                               int64_t T, int64_t d_in, int64_t d_out, int r, void *stream);

/*
 * Multi-envelope form of the two calls above (Eq. 4, ell >= 1), dense rows: s_in is ell x d_in,
 * s_r ell x r, s_out ell x d_out.  dtype: LORDBA_BF16, LORDBA_F16 or LORDBA_F32.
 */
int lordba_adapter_forward_ell(const void *x, const uint32_t *packed_A, const uint32_t *packed_B,
                               const float *s_in, const float *s_r, const float *s_out, void *y,
                               int64_t T, int64_t d_in, int64_t d_out, int r, int ell, int dtype,
                               void *stream);

/* Same operation with explicit row pitches and dtype.  p: [host]. */
int lordba_adapter_forward_ex(const lordba_proj *p, int64_t T, int dtype, void *stream);

/*
 * The adapter forward of n_proj projections that share T and dtype (for
 * instance the seven adapted projections q,k,v,o,gate,up,down of one decoder
 * layer, Section 5 Setup) in as few launches as the kernel-parameter space
 * allows.  projs: [host] array, read before the call returns.  The projections
 * are treated as simultaneous: their y buffers must be pairwise disjoint and no
 * projection's x may overlap any projection's y (LORDBA_EINVAL otherwise); the
 * launches of one call may therefore overlap on the GPU.
 */
int lordba_adapter_forward_batched(const lordba_proj *projs, int n_proj, int64_t T, int dtype,
                                   void *stream);

/*
 * Multi-adapter batch (Section 2, adapter-mode deployment, condition A4: many task adapters
 * served over one frozen base): segment i is tokens[i] consecutive token rows that go through their own adapter.
 * segs[i].x / .y point at the segment's first row (usually into one shared x / y matrix),
 * the other fields name the segment's adapter; several segments may share an adapter.
 * segs, tokens: [host] arrays of n_seg entries, read before the call returns.  Segments are
 * treated as simultaneous (same disjointness rules as the batched call); empty segments are
 * skipped.  One launch per 24 segments of equal padded rank (per 96 on the tcgen05 kernel).
 */
int lordba_adapter_forward_segments(const lordba_proj *segs, const int64_t *tokens, int n_seg, int dtype,
                                    void *stream);

/*
 * Host-buffer form of lordba_adapter_forward{,_f32}: x_host and y_host are
 * [host] (pinned memory makes the copies asynchronous), dense rows; the carriers
 * and scales stay [device] because they are loaded once per adapter.
 * workspace: [device], at least lordba_host_workspace_bytes() bytes, 256-byte
 * aligned.  Enqueues H2D(x), H2D(y), the forward kernel and D2H(y) on `stream`;
 * y_host is valid once the stream has been synchronised.
 */
size_t lordba_host_workspace_bytes(int64_t T, int64_t d_in, int64_t d_out, int dtype);
int lordba_adapter_forward_host(const void *x_host, const uint32_t *packed_A,
                                const uint32_t *packed_B, const float *s_in, const float *s_r,
                                const float *s_out, void *y_host, int64_t T, int64_t d_in,
                                int64_t d_out, int r, int dtype, void *workspace,
                                size_t workspace_bytes, void *stream);

/*
 * lordba_adapter_forward_host without a caller-supplied workspace (an addition of this library;
 * the paper has no counterpart).
 *
 * For callers that have host activations but are not in a position to obtain device memory: code
 * that runs where cudaMalloc is off limits (inside a latency-critical loop, since an allocation
 * can synchronise the whole device; under a host framework that owns all device memory and hands
 * none to plug-ins; in a process whose memory budget was fixed at start-up).  The device staging
 * area for x and y is a buffer of LORDBA_STATIC_SCRATCH_BYTES that is part of the library image:
 * every GPU on which the library is loaded holds it until the process exits, and this call
 * allocates nothing and frees nothing.
 *
 *   - Same arguments, order of work and result as lordba_adapter_forward_host, minus the
 *     workspace.  If lordba_host_workspace_bytes(T, d_in, d_out, dtype) exceeds
 *     LORDBA_STATIC_SCRATCH_BYTES the call returns LORDBA_ETOOLARGE and does nothing.
 *   - The first call on a device looks up the buffer's device address (with that device current)
 *     and remembers it.  If nothing of the library has run on that device yet, this lookup is
 *     also the moment at which the CUDA runtime loads the library's device code there, which
 *     reserves the buffer and may synchronise the device: make that first call at start-up,
 *     outside any stream capture and outside latency-critical code.
 *   - All calls on a device share the one buffer.  It still holds the previous call's x and y;
 *     nothing in it has to start at zero, because every byte that is read was copied in by the
 *     same call first.  Two calls whose work overlaps on the GPU (different streams, no
 *     ordering between them) would overwrite each other's staging data: order them.
 */
#define LORDBA_STATIC_SCRATCH_BYTES (8u << 20)
int lordba_adapter_forward_host_static(const void *x_host, const uint32_t *packed_A,
                                       const uint32_t *packed_B, const float *s_in, const float *s_r,
                                       const float *s_out, void *y_host, int64_t T, int64_t d_in,
                                       int64_t d_out, int r, int dtype, void *stream);

/*
 * Which kernel family a call would run each projection on, without launching anything: the
 * answer of lordba_adapter_forward_batched (tokens == NULL: every projection has T rows) or of
 * lordba_adapter_forward_segments (tokens[i] rows each) for the same arguments and the current
 * lordba_set_variant setting.  variants: [host] n_proj entries, each set to LORDBA_VARIANT_FMA,
 * _TC or _MMA (0 for a projection without rows).  The CUDA-core kernel (FMA) takes every shape but
 * runs an order of magnitude below the tensor-core kernels, which want bf16 / float16 activations,
 * d_in and d_out multiples of 64, row pitches multiples of 8 elements and 16-byte aligned x, y,
 * scales and carriers: a caller can see that fallback coming here.  Returns the status the call
 * itself would return for bad arguments.
 */
int lordba_query_variant(const lordba_proj *projs, int n_proj, int64_t T, const int64_t *tokens, int dtype,
                         int *variants);

/*
 * Prepared calls.  Every forward call builds its launch parameters on the host first (tensor maps
 * for the copy engine, six per projection in the streaming kernel).  A caller that repeats a call
 * with the same pointers and sizes (a layer's adapters over fixed activation buffers, step after
 * step) can have that done once:
 *
 *   lordba_plan_bytes   the storage a plan for these arguments needs (0 on bad arguments);
 *   lordba_plan_init    validates the arguments exactly like lordba_adapter_forward_batched
 *                       (tokens == NULL) or lordba_adapter_forward_segments (tokens given), chooses
 *                       the kernels and writes the prepared launches into plan: [host], 64-byte
 *                       aligned, caller-owned, plan_bytes long (LORDBA_ETOOLARGE if too short).
 *                       Nothing is launched;
 *   lordba_adapter_forward_planned   enqueues the prepared launches on stream: the same kernels
 *                       with the same arguments as the unprepared call.
 *
 * A plan holds device addresses: it belongs to the device that was current at lordba_plan_init
 * (LORDBA_EINVAL on another one), stays valid while the buffers it names are, and may be replayed
 * any number of times, from any stream; it holds no resources and needs no release.
 * LORDBA_PROJ_OVERLAP and LORDBA_PROJ_X_READY in the projections' flags are part of the plan.
 */
size_t lordba_plan_bytes(const lordba_proj *projs, int n_proj, int64_t T, const int64_t *tokens, int dtype);
int lordba_plan_init(void *plan, size_t plan_bytes, const lordba_proj *projs, int n_proj, int64_t T,
                     const int64_t *tokens, int dtype);
int lordba_adapter_forward_planned(const void *plan, void *stream);
/* Kernel launches a plan holds (-1 if plan is not a plan). */
int lordba_plan_launches(const void *plan);

/*
 * Closed-form scale updates of the adapter fit (Appendix "Closed-form scale updates for
 * PTQ-LoRDBA"; the scale step Eq. scales-step of the PTQ-LoRDBA iteration, and the sweep that
 * initialises the scales after the SVD warm start, Eq. svd-init).  With the packed carriers held
 * fixed, `sweeps` block-coordinate sweeps of
 *
 *     min  1/2 || target - diag(s_in) A_sign^T diag(s_r) B_sign^T diag(s_out) ||_F^2
 *
 * each sweep updating s_in (Eq. alpha-update: one scalar least squares per row of the target), then
 * s_r (Eq. beta-gram and Eq. beta-pinv: the r x r normal equations G = (P^T P) o (Q Q^T), solved
 * by the Moore-Penrose pseudo-inverse, eigenvalues below r * 2^-52 * lambda_max dropped), then
 * s_out (Eq. gamma-update: one scalar least squares per column); a row or column whose model is
 * identically zero gets 0.  axes: which of the three a sweep updates (LORDBA_FIT_ALPHA | _BETA |
 * _GAMMA; LORDBA_FIT_ALL for the full sweep), always in that order.
 *
 * target: [device] float32, d_in x d_out row-major with row pitch ld >= d_out elements (the dense
 * adapter Delta-W* that is being fitted, in the orientation y = x Delta-W); read only.  packed_A,
 * packed_B: the carriers as lordba_pack_signs makes them.  s_in (d_in), s_r (r), s_out (d_out):
 * [device] float32, read as the starting point and overwritten with the result.  workspace:
 * [device], 256-byte aligned, at least lordba_fit_workspace_bytes() bytes (LORDBA_EINVAL if
 * shorter); its contents need not be initialised and are not meaningful afterwards.  The passes
 * over the target accumulate in float32, everything of size r x r and the quotients in float64;
 * results are deterministic.  Asynchronous on stream; sweeps = 0 is a no-op.
 */
#define LORDBA_FIT_ALPHA 1
#define LORDBA_FIT_BETA 2
#define LORDBA_FIT_GAMMA 4
#define LORDBA_FIT_ALL 7
size_t lordba_fit_workspace_bytes(int64_t d_in, int64_t d_out, int r);
int lordba_fit_scales(const float *target, int64_t ld, const uint32_t *packed_A, const uint32_t *packed_B,
                      float *s_in, float *s_r, float *s_out, int64_t d_in, int64_t d_out, int r, int sweeps,
                      int axes, void *workspace, size_t workspace_bytes, void *stream);

/* Storage of one adapter in bits, Eq. 5: r(d_in+d_out) + 16 ell (d_in+r+d_out). */
int64_t lordba_adapter_bits(int64_t d_in, int64_t d_out, int r, int ell);

/* Pin the kernel family used by the forward entry points (process-wide). */
int lordba_set_variant(int variant);
int lordba_get_variant(void);

/*
 * Bounded device-side waits (TMA / MMA completion barriers) record a non-zero
 * code in a device status word instead of spinning forever.  This call
 * synchronises `stream`, copies the word to *code, clears it, and returns
 * LORDBA_ETIMEOUT if it was non-zero.
 */
int lordba_device_status(int *code, void *stream);

/* Kernels launched by this library in this process so far. */
int64_t lordba_launch_count(void);

const char *lordba_status_string(int status);
const char *lordba_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LORDBA_H_ */
