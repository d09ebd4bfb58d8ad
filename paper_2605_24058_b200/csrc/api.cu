// C ABI of liblordba: argument validation on the host, kernel-family choice,
// launches.  See include/lordba.h for the contract of every entry point.
#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "lordba_internal.h"

namespace lordba {

namespace {
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_variant{LORDBA_VARIANT_AUTO};
__device__ int g_device_status;   // written by bounded waits that gave up
std::mutex g_status_mutex;
int *g_status_ptr[64] = {nullptr};
#ifdef LORDBA_TEST_HOOKS
std::atomic<int> g_test_skip_item{-1};
#endif
}  // namespace

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int *device_status_word()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_status_mutex);
    if (!g_status_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        g_status_ptr[dev] = static_cast<int *>(p);
    }
    return g_status_ptr[dev];
}

int test_skip_item()
{
#ifdef LORDBA_TEST_HOOKS
    return g_test_skip_item.load(std::memory_order_relaxed);
#else
    return -1;
#endif
}

int FamilySelector::family(const lordba_proj &p, int64_t rows) const
{
    if (rows <= 0) return 0;
    if (variant == LORDBA_VARIANT_FMA || dtype == LORDBA_F32) return LORDBA_VARIANT_FMA;
    if (use_tc) return tc_supported(p, rows, dtype) ? LORDBA_VARIANT_TC : LORDBA_VARIANT_FMA;
    if (mma_supported(p, rows, dtype)) return LORDBA_VARIANT_MMA;
    // Left to itself the library also gives the tcgen05 kernel what the streaming kernel cannot take
    // but it can (widths that are not multiples of 64), from one 128-token tile up: a fifth to a
    // half of the roofline there instead of the CUDA-core kernel's tenth.
    if (variant == LORDBA_VARIANT_AUTO && rows >= 128 && tc_supported(p, rows, dtype)) return LORDBA_VARIANT_TC;
    return LORDBA_VARIANT_FMA;
}

int launch_record(const LaunchRec &rec, const void *arg0, const void *arg1, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(rec.grid[0], rec.grid[1], rec.grid[2]);
    cfg.blockDim = dim3(rec.block, 1, 1);
    cfg.dynamicSmemBytes = rec.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned na = 0;
    if (rec.cluster > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = rec.cluster_z ? 1 : rec.cluster; attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = rec.cluster_z ? rec.cluster : 1;
        ++na;
    }
    if (rec.pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    void *args[2] = {const_cast<void *>(arg0), const_cast<void *>(arg1)};
    if (cudaLaunchKernelExC(&cfg, rec.func, args) != cudaSuccess) {
        cudaGetLastError();
        return LORDBA_ECUDA;
    }
    count_launch();
    return LORDBA_OK;
}

int LaunchSink::emit(LaunchRec rec, const void *arg0, const void *arg1)
{
    if (immediate) return launch_record(rec, arg0, arg1, stream);
    const size_t a0 = (sizeof(LaunchRec) + 63) / 64 * 64;
    const size_t a1 = a0 + ((size_t)rec.arg_bytes[0] + 63) / 64 * 64;
    const size_t total = a1 + (rec.n_args > 1 ? ((size_t)rec.arg_bytes[1] + 63) / 64 * 64 : 0);
    rec.total_bytes = (uint32_t)total;
    if (buf) {
        if (used + total > cap) return LORDBA_ETOOLARGE;
        std::memcpy(buf + used, &rec, sizeof(rec));
        std::memcpy(buf + used + a0, arg0, rec.arg_bytes[0]);
        if (rec.n_args > 1) std::memcpy(buf + used + a1, arg1, rec.arg_bytes[1]);
    }
    used += total;
    ++count;
    return LORDBA_OK;
}

namespace {

bool aligned(const void *p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; }

bool overlaps(const void *a, size_t na, const void *b, size_t nb)
{
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + nb && b0 < a0 + na;
}

bool known_dtype(int dtype) { return dtype == LORDBA_F32 || dtype == LORDBA_BF16 || dtype == LORDBA_F16; }

int validate_proj(const lordba_proj &p, int64_t T, int dtype)
{
    if (!known_dtype(dtype)) return LORDBA_EUNSUPPORTED;
    if (T < 0 || p.d_in < 1 || p.d_out < 1 || p.ldx < p.d_in || p.ldy < p.d_out) return LORDBA_EINVAL;
    if ((p.flags & ~(LORDBA_PROJ_OVERLAP | LORDBA_PROJ_SCALES_F16 | LORDBA_PROJ_X_READY | 0xf00)) != 0) return LORDBA_EINVAL;
    if (((p.flags >> 8) & 0xf) + 1 > LORDBA_MAX_ELL) return LORDBA_EUNSUPPORTED;
    if (p.r < 1 || p.r > kMaxRank) return LORDBA_EUNSUPPORTED;
    if (T == 0) return LORDBA_OK;   // nothing is touched: the pointers may be anything
    if (!p.x || !p.packed_A || !p.packed_B || !p.s_in || !p.s_r || !p.s_out || !p.y)
        return LORDBA_EINVAL;
    const size_t e = (dtype == LORDBA_F32) ? 4 : 2;
    if (!aligned(p.x, e) || !aligned(p.y, e) || !aligned(p.packed_A, 4) || !aligned(p.packed_B, 4) ||
        !aligned(p.s_in, 4) || !aligned(p.s_r, 4) || !aligned(p.s_out, 4))
        return LORDBA_EALIGN;
    if (T > 0) {
        const size_t nx = ((size_t)(T - 1) * p.ldx + p.d_in) * e;
        const size_t ny = ((size_t)(T - 1) * p.ldy + p.d_out) * e;
        if (overlaps(p.x, nx, p.y, ny)) return LORDBA_EINVAL;
    }
    return LORDBA_OK;
}

// Left to itself the library takes the tcgen05 kernel where it was measured ahead of the
// streaming one: ranks above 32 from 32 tiles of 128 tokens (one projection at T = 4096, a layer
// at T = 2048), ranks 24 and 32 from eight waves of such tiles (below that the streaming kernel
// is ahead).
FamilySelector make_selector(const lordba_proj *projs, int n, int64_t T, const int64_t *tokens, int dtype)
{
    FamilySelector sel;
    sel.dtype = dtype;
    sel.variant = g_variant.load(std::memory_order_relaxed);
    sel.use_tc = (sel.variant == LORDBA_VARIANT_TC);
    if (sel.variant == LORDBA_VARIANT_AUTO && dtype != LORDBA_F32) {
        int64_t tiles = 0;
        bool all_ok = false, all_high = true;
        for (int i = 0; i < n; ++i) {
            const int64_t rows = rows_of(tokens, T, i);
            if (rows == 0) continue;
            if (tiles == 0) all_ok = true;
            // (what counts is the width of the intermediate: envelopes x rank)
            const int width = (((projs[i].flags >> 8) & 0xf) + 1) * projs[i].r;
            all_ok = all_ok && width > 16 && tc_supported(projs[i], rows, dtype);
            all_high = all_high && width > 32;
            tiles += (rows + 127) / 128;
        }
        sel.use_tc = all_ok && tiles >= (all_high ? 32 : 8 * 148);
    }
    return sel;
}

// batch_checked: the caller has verified that the projections of this call are independent of
// one another (disjoint y buffers, no x inside a y), so its launches may overlap each other.
// tokens: per-projection token rows, or nullptr when every projection has T rows.
int dispatch(const lordba_proj *projs, int n, int64_t T, const int64_t *tokens, int dtype, LaunchSink &sink,
             bool batch_checked)
{
    const FamilySelector sel = make_selector(projs, n, T, tokens, dtype);
    if (sel.variant != LORDBA_VARIANT_AUTO) {
        // a pinned family must be able to take every projection of the call
        for (int i = 0; i < n; ++i) {
            const int64_t rows = rows_of(tokens, T, i);
            if (rows > 0 && sel.family(projs[i], rows) != sel.variant) return LORDBA_EUNSUPPORTED;
        }
    }
    int launches = 0;
    int rc = launch_forward_tc(projs, tokens, T, n, sel, sink, batch_checked, &launches);
    if (rc != LORDBA_OK) return rc;
    rc = launch_forward_mma(projs, tokens, T, n, sel, sink, batch_checked, &launches);
    if (rc != LORDBA_OK) return rc;
    return launch_forward_fma(projs, tokens, T, n, sel, sink);
}

int dispatch_now(const lordba_proj *projs, int n, int64_t T, const int64_t *tokens, int dtype, cudaStream_t stream,
                 bool batch_checked)
{
    LaunchSink sink;
    sink.stream = stream;
    return dispatch(projs, n, T, tokens, dtype, sink, batch_checked);
}

size_t bytes_of(const lordba_proj &p, int64_t rows, int64_t ld, int64_t width, size_t e)
{
    (void)p;
    return ((size_t)(rows - 1) * (size_t)ld + (size_t)width) * e;
}

// The projections of a call are simultaneous: outputs pairwise disjoint, no input inside an
// output.  Sorted intervals: n log n.
int check_independent(const lordba_proj *projs, int n, int64_t T, const int64_t *tokens, size_t e)
{
    struct Iv { uintptr_t lo, hi; };
    Iv ys[kMaxCallProjs];
    int m = 0;
    for (int i = 0; i < n; ++i) {
        const int64_t rows = rows_of(tokens, T, i);
        if (rows <= 0) continue;
        const uintptr_t lo = reinterpret_cast<uintptr_t>(projs[i].y);
        ys[m++] = Iv{lo, lo + bytes_of(projs[i], rows, projs[i].ldy, projs[i].d_out, e)};
    }
    std::sort(ys, ys + m, [](const Iv &a, const Iv &b) { return a.lo < b.lo; });
    for (int i = 0; i + 1 < m; ++i)
        if (ys[i].hi > ys[i + 1].lo) return LORDBA_EINVAL;
    for (int i = 0; i < n; ++i) {
        const int64_t rows = rows_of(tokens, T, i);
        if (rows <= 0) continue;
        const uintptr_t lo = reinterpret_cast<uintptr_t>(projs[i].x);
        const uintptr_t hi = lo + bytes_of(projs[i], rows, projs[i].ldx, projs[i].d_in, e);
        // first output that ends after the input starts (the outputs are disjoint: their ends are sorted too)
        const Iv *it = std::upper_bound(ys, ys + m, lo, [](uintptr_t v, const Iv &a) { return v < a.hi; });
        if (it != ys + m && it->lo < hi) return LORDBA_EINVAL;
    }
    return LORDBA_OK;
}

// Validation shared by the batched, the segmented and the prepared calls.
int validate_call(const lordba_proj *projs, int n, int64_t T, const int64_t *tokens, int dtype)
{
    if (n < 0 || (n > 0 && !projs)) return LORDBA_EINVAL;
    if (n > kMaxCallProjs) return LORDBA_EUNSUPPORTED;
    if (!tokens && T < 0) return LORDBA_EINVAL;
    for (int i = 0; i < n; ++i) {
        const int rc = validate_proj(projs[i], rows_of(tokens, T, i), dtype);
        if (rc != LORDBA_OK) return rc;
    }
    return check_independent(projs, n, T, tokens, (dtype == LORDBA_F32) ? 4 : 2);
}

lordba_proj dense_proj(const void *x, const uint32_t *pa, const uint32_t *pb, const float *s_in,
                       const float *s_r, const float *s_out, void *y, int64_t d_in, int64_t d_out, int r)
{
    lordba_proj p;
    std::memset(&p, 0, sizeof(p));
    p.x = x; p.packed_A = pa; p.packed_B = pb; p.s_in = s_in; p.s_r = s_r; p.s_out = s_out; p.y = y;
    p.d_in = d_in; p.d_out = d_out; p.ldx = d_in; p.ldy = d_out; p.r = r;
    return p;
}

}  // namespace
}  // namespace lordba

using namespace lordba;

extern "C" {

int64_t lordba_packed_words(int64_t rows, int64_t cols, int role)
{
    if (rows < 0 || cols < 0) return -1;
    if (role == 0) return ((cols + 63) / 64) * rows * 2;
    if (role == 1) return (rows * cols + 31) / 32;
    return -1;
}

int lordba_pack_signs(const int8_t *signs, int64_t rows, int64_t cols, int role, uint32_t *packed,
                      void *stream)
{
    if (role != 0 && role != 1) return LORDBA_EUNSUPPORTED;
    if (rows < 0 || cols < 0) return LORDBA_EINVAL;
    if (rows == 0 || cols == 0) return LORDBA_OK;
    if (!signs || !packed) return LORDBA_EINVAL;
    if (!aligned(packed, 4)) return LORDBA_EALIGN;
    return launch_pack(signs, rows, cols, role, packed, static_cast<cudaStream_t>(stream));
}

int lordba_scales_from_f16(const uint16_t *src, float *dst, int64_t n, void *stream)
{
    if (n < 0) return LORDBA_EINVAL;
    if (n == 0) return LORDBA_OK;
    if (!src || !dst) return LORDBA_EINVAL;
    if (!aligned(src, 2) || !aligned(dst, 4)) return LORDBA_EALIGN;
    return launch_widen_scales(src, dst, n, static_cast<cudaStream_t>(stream));
}

int lordba_unpack_signs(const uint32_t *packed, int64_t rows, int64_t cols, int role, int8_t *signs,
                        void *stream)
{
    if (role != 0 && role != 1) return LORDBA_EUNSUPPORTED;
    if (rows < 0 || cols < 0) return LORDBA_EINVAL;
    if (rows == 0 || cols == 0) return LORDBA_OK;
    if (!signs || !packed) return LORDBA_EINVAL;
    if (!aligned(packed, 4)) return LORDBA_EALIGN;
    return launch_unpack(packed, rows, cols, role, signs, static_cast<cudaStream_t>(stream));
}

int lordba_adapter_forward_ex(const lordba_proj *p, int64_t T, int dtype, void *stream)
{
    if (!p) return LORDBA_EINVAL;
    const int rc = validate_proj(*p, T, dtype);
    if (rc != LORDBA_OK) return rc;
    if (T == 0) return LORDBA_OK;
    return dispatch_now(p, 1, T, nullptr, dtype, static_cast<cudaStream_t>(stream), false);
}

int lordba_adapter_forward(const void *x, const uint32_t *packed_A, const uint32_t *packed_B,
                           const float *s_in, const float *s_r, const float *s_out, void *y,
                           int64_t T, int64_t d_in, int64_t d_out, int r, void *stream)
{
    const lordba_proj p = dense_proj(x, packed_A, packed_B, s_in, s_r, s_out, y, d_in, d_out, r);
    return lordba_adapter_forward_ex(&p, T, LORDBA_BF16, stream);
}

int lordba_adapter_forward_ell(const void *x, const uint32_t *packed_A, const uint32_t *packed_B,
                               const float *s_in, const float *s_r, const float *s_out, void *y,
                               int64_t T, int64_t d_in, int64_t d_out, int r, int ell, int dtype,
                               void *stream)
{
    if (ell < 1 || ell > LORDBA_MAX_ELL) return LORDBA_EUNSUPPORTED;
    lordba_proj p = dense_proj(x, packed_A, packed_B, s_in, s_r, s_out, y, d_in, d_out, r);
    p.flags = LORDBA_PROJ_ELL(ell);
    return lordba_adapter_forward_ex(&p, T, dtype, stream);
}

int lordba_adapter_forward_f32(const float *x, const uint32_t *packed_A, const uint32_t *packed_B,
                               const float *s_in, const float *s_r, const float *s_out, float *y,
                               int64_t T, int64_t d_in, int64_t d_out, int r, void *stream)
{
    const lordba_proj p = dense_proj(x, packed_A, packed_B, s_in, s_r, s_out, y, d_in, d_out, r);
    return lordba_adapter_forward_ex(&p, T, LORDBA_F32, stream);
}

int lordba_adapter_forward_batched(const lordba_proj *projs, int n_proj, int64_t T, int dtype,
                                   void *stream)
{
    const int rc = validate_call(projs, n_proj, T, nullptr, dtype);
    if (rc != LORDBA_OK) return rc;
    if (T == 0 || n_proj == 0) return LORDBA_OK;
    return dispatch_now(projs, n_proj, T, nullptr, dtype, static_cast<cudaStream_t>(stream), true);
}

int lordba_adapter_forward_segments(const lordba_proj *segs, const int64_t *tokens, int n_seg, int dtype,
                                    void *stream)
{
    if (n_seg > 0 && !tokens) return LORDBA_EINVAL;
    const int rc = validate_call(segs, n_seg, 0, tokens, dtype);
    if (rc != LORDBA_OK) return rc;
    if (n_seg == 0) return LORDBA_OK;
    return dispatch_now(segs, n_seg, 0, tokens, dtype, static_cast<cudaStream_t>(stream), true);
}

int lordba_query_variant(const lordba_proj *projs, int n_proj, int64_t T, const int64_t *tokens, int dtype,
                         int *variants)
{
    if (!variants && n_proj > 0) return LORDBA_EINVAL;
    const int rc = validate_call(projs, n_proj, T, tokens, dtype);
    if (rc != LORDBA_OK) return rc;
    const FamilySelector sel = make_selector(projs, n_proj, T, tokens, dtype);
    for (int i = 0; i < n_proj; ++i) {
        const int64_t rows = rows_of(tokens, T, i);
        variants[i] = sel.family(projs[i], rows);
        if (rows > 0 && sel.variant != LORDBA_VARIANT_AUTO && variants[i] != sel.variant) return LORDBA_EUNSUPPORTED;
    }
    return LORDBA_OK;
}

// ---- prepared calls -----------------------------------------------------------------------

namespace {
struct PlanHeader {
    uint32_t magic, version;
    int32_t device;
    int32_t n_launches;
    uint64_t bytes;        // header + records
    uint64_t pad_[5];
};
static_assert(sizeof(PlanHeader) == 64, "plan header is one 64-byte block");
constexpr uint32_t kPlanMagic = 0x4c44424du, kPlanVersion = 2;

int build_plan(void *storage, size_t cap, const lordba_proj *projs, int n_proj, int64_t T, const int64_t *tokens,
               int dtype, size_t *bytes_out)
{
    const int rc = validate_call(projs, n_proj, T, tokens, dtype);
    if (rc != LORDBA_OK) return rc;
    LaunchSink sink;
    sink.immediate = false;
    if (storage) {
        if (!aligned(storage, 64)) return LORDBA_EALIGN;
        if (cap < sizeof(PlanHeader)) return LORDBA_ETOOLARGE;
        sink.buf = static_cast<uint8_t *>(storage) + sizeof(PlanHeader);
        sink.cap = cap - sizeof(PlanHeader);
    }
    bool any = false;
    for (int i = 0; i < n_proj; ++i) any = any || rows_of(tokens, T, i) > 0;
    if (any) {
        const int rc2 = dispatch(projs, n_proj, T, tokens, dtype, sink, true);
        if (rc2 != LORDBA_OK) return rc2;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LORDBA_ECUDA;
    if (storage) {
        PlanHeader h;
        std::memset(&h, 0, sizeof(h));
        h.magic = kPlanMagic; h.version = kPlanVersion; h.device = dev; h.n_launches = sink.count;
        h.bytes = sizeof(PlanHeader) + sink.used;
        std::memcpy(storage, &h, sizeof(h));
    }
    if (bytes_out) *bytes_out = sizeof(PlanHeader) + sink.used;
    return LORDBA_OK;
}
}  // namespace

size_t lordba_plan_bytes(const lordba_proj *projs, int n_proj, int64_t T, const int64_t *tokens, int dtype)
{
    size_t bytes = 0;
    if (build_plan(nullptr, 0, projs, n_proj, T, tokens, dtype, &bytes) != LORDBA_OK) return 0;
    return bytes;
}

int lordba_plan_init(void *plan, size_t plan_bytes, const lordba_proj *projs, int n_proj, int64_t T,
                     const int64_t *tokens, int dtype)
{
    if (!plan) return LORDBA_EINVAL;
    return build_plan(plan, plan_bytes, projs, n_proj, T, tokens, dtype, nullptr);
}

int lordba_plan_launches(const void *plan)
{
    if (!plan || !aligned(plan, 64)) return -1;
    const PlanHeader *h = static_cast<const PlanHeader *>(plan);
    if (h->magic != kPlanMagic || h->version != kPlanVersion) return -1;
    return h->n_launches;
}

int lordba_adapter_forward_planned(const void *plan, void *stream)
{
    if (!plan) return LORDBA_EINVAL;
    if (!aligned(plan, 64)) return LORDBA_EALIGN;
    const PlanHeader *h = static_cast<const PlanHeader *>(plan);
    if (h->magic != kPlanMagic || h->version != kPlanVersion) return LORDBA_EINVAL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return LORDBA_ECUDA;
    if (dev != h->device) return LORDBA_EINVAL;      // a plan holds addresses of the device it was made on
    const uint8_t *p = static_cast<const uint8_t *>(plan) + sizeof(PlanHeader);
    const uint8_t *end = static_cast<const uint8_t *>(plan) + h->bytes;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int i = 0; i < h->n_launches; ++i) {
        const LaunchRec *rec = reinterpret_cast<const LaunchRec *>(p);
        if (p + sizeof(LaunchRec) > end || p + rec->total_bytes > end) return LORDBA_EINVAL;
        const size_t a0 = (sizeof(LaunchRec) + 63) / 64 * 64;
        const size_t a1 = a0 + ((size_t)rec->arg_bytes[0] + 63) / 64 * 64;
        const int rc = launch_record(*rec, p + a0, rec->n_args > 1 ? p + a1 : nullptr, s);
        if (rc != LORDBA_OK) return rc;
        p += rec->total_bytes;
    }
    return LORDBA_OK;
}

#ifdef LORDBA_TEST_HOOKS
// Test-hooks build only: the producers of the tensor-core kernels leave out the copy request of
// pipeline item `item` (counted from 0 within every CTA's first tile); -1 switches the hook off.
int lordba_test_skip_item(int item)
{
    g_test_skip_item.store(item, std::memory_order_relaxed);
    return LORDBA_OK;
}
#endif

size_t lordba_host_workspace_bytes(int64_t T, int64_t d_in, int64_t d_out, int dtype)
{
    if (T < 0 || d_in < 0 || d_out < 0) return 0;
    const size_t e = (dtype == LORDBA_F32) ? 4 : 2;
    const size_t nx = ((size_t)T * d_in * e + 255) / 256 * 256;
    const size_t ny = ((size_t)T * d_out * e + 255) / 256 * 256;
    return nx + ny;
}

int lordba_adapter_forward_host(const void *x_host, const uint32_t *packed_A,
                                const uint32_t *packed_B, const float *s_in, const float *s_r,
                                const float *s_out, void *y_host, int64_t T, int64_t d_in,
                                int64_t d_out, int r, int dtype, void *workspace,
                                size_t workspace_bytes, void *stream)
{
    if (!known_dtype(dtype)) return LORDBA_EUNSUPPORTED;
    if (T < 0 || d_in < 1 || d_out < 1) return LORDBA_EINVAL;
    if (!x_host || !y_host || !workspace) return LORDBA_EINVAL;
    if (!aligned(workspace, 256)) return LORDBA_EALIGN;
    if (workspace_bytes < lordba_host_workspace_bytes(T, d_in, d_out, dtype)) return LORDBA_EINVAL;
    const size_t e = (dtype == LORDBA_F32) ? 4 : 2;
    const size_t bx = (size_t)T * d_in * e, by = (size_t)T * d_out * e;
    char *xd = static_cast<char *>(workspace);
    char *yd = xd + (bx + 255) / 256 * 256;
    const lordba_proj p = dense_proj(xd, packed_A, packed_B, s_in, s_r, s_out, yd, d_in, d_out, r);
    const int rc = validate_proj(p, T, dtype);
    if (rc != LORDBA_OK) return rc;
    if (T == 0) return LORDBA_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(xd, x_host, bx, cudaMemcpyHostToDevice, s) != cudaSuccess) return LORDBA_ECUDA;
    if (cudaMemcpyAsync(yd, y_host, by, cudaMemcpyHostToDevice, s) != cudaSuccess) return LORDBA_ECUDA;
    const int rc2 = dispatch_now(&p, 1, T, nullptr, dtype, s, false);
    if (rc2 != LORDBA_OK) return rc2;
    if (cudaMemcpyAsync(y_host, yd, by, cudaMemcpyDeviceToHost, s) != cudaSuccess) return LORDBA_ECUDA;
    return LORDBA_OK;
}

}  // extern "C"

namespace lordba {
namespace {

// Staging area of lordba_adapter_forward_host_static.  In host code this name is only a handle
// for cudaGetSymbolAddress, never a pointer that a kernel or a copy could use.
static __device__ __align__(256) unsigned char g_static_scratch[LORDBA_STATIC_SCRATCH_BYTES];
std::mutex g_scratch_mutex;
void *g_scratch_ptr[64] = {nullptr};

// Device address of the staging area on the current device (looked up once per device).
void *static_scratch()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        g_scratch_ptr[dev] = p;
    }
    return g_scratch_ptr[dev];
}

}  // namespace
}  // namespace lordba

extern "C" {

int lordba_adapter_forward_host_static(const void *x_host, const uint32_t *packed_A,
                                       const uint32_t *packed_B, const float *s_in, const float *s_r,
                                       const float *s_out, void *y_host, int64_t T, int64_t d_in,
                                       int64_t d_out, int r, int dtype, void *stream)
{
    if (!known_dtype(dtype)) return LORDBA_EUNSUPPORTED;
    if (T < 0 || d_in < 1 || d_out < 1) return LORDBA_EINVAL;
    const size_t e = (dtype == LORDBA_F32) ? 4 : 2;
    // sizes that cannot fit are refused before any multiplication can overflow
    const size_t limit = LORDBA_STATIC_SCRATCH_BYTES;
    if ((size_t)T > limit || (size_t)d_in > limit || (size_t)d_out > limit ||
        (size_t)T * (size_t)(d_in + d_out) > limit / e)
        return LORDBA_ETOOLARGE;
    const size_t need = lordba_host_workspace_bytes(T, d_in, d_out, dtype);
    if (need > limit) return LORDBA_ETOOLARGE;
    void *scratch = static_scratch();
    if (!scratch) return LORDBA_ECUDA;
    return lordba_adapter_forward_host(x_host, packed_A, packed_B, s_in, s_r, s_out, y_host, T, d_in,
                                       d_out, r, dtype, scratch, limit, stream);
}

size_t lordba_fit_workspace_bytes(int64_t d_in, int64_t d_out, int r)
{
    if (d_in < 1 || d_out < 1 || r < 1 || r > kMaxRank) return 0;
    return fit_workspace_bytes(d_in, d_out, r);
}

int lordba_fit_scales(const float *target, int64_t ld, const uint32_t *packed_A, const uint32_t *packed_B,
                      float *s_in, float *s_r, float *s_out, int64_t d_in, int64_t d_out, int r, int sweeps,
                      int axes, void *workspace, size_t workspace_bytes, void *stream)
{
    if (r < 1 || r > kMaxRank) return LORDBA_EUNSUPPORTED;
    if (d_in < 1 || d_out < 1 || ld < d_out || sweeps < 0) return LORDBA_EINVAL;
    if (axes < 1 || axes > LORDBA_FIT_ALL) return LORDBA_EINVAL;
    if (!target || !packed_A || !packed_B || !s_in || !s_r || !s_out || !workspace) return LORDBA_EINVAL;
    if (!aligned(target, 4) || !aligned(packed_A, 4) || !aligned(packed_B, 4) || !aligned(s_in, 4) ||
        !aligned(s_r, 4) || !aligned(s_out, 4) || !aligned(workspace, 256))
        return LORDBA_EALIGN;
    if (workspace_bytes < fit_workspace_bytes(d_in, d_out, r)) return LORDBA_EINVAL;
    if (sweeps == 0) return LORDBA_OK;
    return launch_fit_scales(target, ld, packed_A, packed_B, s_in, s_r, s_out, d_in, d_out, r, sweeps, axes,
                             workspace, static_cast<cudaStream_t>(stream));
}

int64_t lordba_adapter_bits(int64_t d_in, int64_t d_out, int r, int ell)
{
    return (int64_t)r * (d_in + d_out) + 16 * (int64_t)ell * (d_in + r + d_out);
}

int lordba_set_variant(int variant)
{
    if (variant < LORDBA_VARIANT_AUTO || variant > LORDBA_VARIANT_MMA) return LORDBA_EUNSUPPORTED;
    g_variant.store(variant, std::memory_order_relaxed);
    return LORDBA_OK;
}

int lordba_get_variant(void) { return g_variant.load(std::memory_order_relaxed); }

int lordba_device_status(int *code, void *stream)
{
    if (!code) return LORDBA_EINVAL;
    int *word = device_status_word();
    if (!word) return LORDBA_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return LORDBA_ECUDA;
    int v = 0;
    if (cudaMemcpy(&v, word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return LORDBA_ECUDA;
    if (v != 0 && cudaMemset(word, 0, sizeof(int)) != cudaSuccess) return LORDBA_ECUDA;
    *code = v;
    return v == 0 ? LORDBA_OK : LORDBA_ETIMEOUT;
}

int64_t lordba_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *lordba_status_string(int status)
{
    switch (status) {
        case LORDBA_OK: return "ok";
        case LORDBA_EINVAL: return "invalid argument";
        case LORDBA_EUNSUPPORTED: return "unsupported rank, dtype, role or variant";
        case LORDBA_EALIGN: return "misaligned pointer";
        case LORDBA_ECUDA: return "CUDA runtime error";
        case LORDBA_ETIMEOUT: return "device-side wait timed out";
        case LORDBA_ETOOLARGE: return "the call needs more than the built-in scratch buffer";
        default: return "unknown status";
    }
}

const char *lordba_version(void) { return "lordba-b200 0.1.0 (sm_100a)"; }

}  // extern "C"
