// C ABI of liblordba: argument validation on the host, kernel-family choice,
// launches.  See include/lordba.h for the contract of every entry point.
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "lordba_internal.h"

namespace lordba {

namespace {
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_variant{LORDBA_VARIANT_AUTO};
__device__ int g_device_status;   // written by bounded waits that gave up
std::mutex g_status_mutex;
int *g_status_ptr[64] = {nullptr};
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
    if ((p.flags & ~(LORDBA_PROJ_OVERLAP | LORDBA_PROJ_SCALES_F16 | 0xf00)) != 0) return LORDBA_EINVAL;
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

// batch_checked: the caller has verified that the projections of this call are independent of
// one another (disjoint y buffers, no x inside a y), so its launches may overlap each other.
// tokens: per-projection token rows, or nullptr when every projection has T rows.
int dispatch(const lordba_proj *projs, int n, int64_t T, const int64_t *tokens, int dtype, cudaStream_t stream,
             bool batch_checked)
{
    const int variant = g_variant.load(std::memory_order_relaxed);
    std::vector<int64_t> rows(n, T);
    if (tokens) rows.assign(tokens, tokens + n);
    if (variant == LORDBA_VARIANT_FMA || dtype == LORDBA_F32) {
        if (variant == LORDBA_VARIANT_TC || variant == LORDBA_VARIANT_MMA) return LORDBA_EUNSUPPORTED;
        return launch_forward_fma(projs, rows.data(), n, dtype, stream);
    }
    // Split the list: what the chosen tensor-core kernel can take, and the rest.  Left to itself
    // the library takes the tcgen05 kernel where it was measured ahead of the streaming one: ranks
    // above 32 from 32 tiles of 128 tokens (one projection at T = 4096, a layer at T = 2048), ranks
    // 24 and 32 from eight waves of such tiles (below that the streaming kernel is ahead).  (That kernel wants one token count for all
    // projections.)
    bool use_tc = (variant == LORDBA_VARIANT_TC);
    if (use_tc && tokens) return LORDBA_EUNSUPPORTED;
    if (variant == LORDBA_VARIANT_AUTO && !tokens) {
        int64_t tiles = 0;
        bool all_ok = n > 0, all_high = true;
        for (int i = 0; i < n; ++i) {
            all_ok = all_ok && projs[i].r > 16 && tc_supported(projs[i], T, dtype);
            all_high = all_high && projs[i].r > 32;
            tiles += T / 128;
        }
        use_tc = all_ok && tiles >= (all_high ? 32 : 8 * 148);
    }
    std::vector<lordba_proj> fast, fma;
    std::vector<int64_t> fast_rows, fma_rows;
    for (int i = 0; i < n; ++i) {
        if (rows[i] == 0) continue;
        const bool ok = use_tc ? tc_supported(projs[i], rows[i], dtype) : mma_supported(projs[i], rows[i], dtype);
        (ok ? fast : fma).push_back(projs[i]);
        (ok ? fast_rows : fma_rows).push_back(rows[i]);
    }
    if (variant != LORDBA_VARIANT_AUTO && !fma.empty()) return LORDBA_EUNSUPPORTED;
    if (!fast.empty()) {
        const int rc = use_tc ? launch_forward_tc(fast.data(), (int)fast.size(), T, dtype, stream, batch_checked)
                              : launch_forward_mma(fast.data(), fast_rows.data(), (int)fast.size(), dtype, stream,
                                                   batch_checked);
        if (rc != LORDBA_OK) return rc;
    }
    if (!fma.empty()) return launch_forward_fma(fma.data(), fma_rows.data(), (int)fma.size(), dtype, stream);
    return LORDBA_OK;
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
    return dispatch(p, 1, T, nullptr, dtype, static_cast<cudaStream_t>(stream), false);
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
    if (n_proj < 0 || (n_proj > 0 && !projs)) return LORDBA_EINVAL;
    const size_t e = (dtype == LORDBA_F32) ? 4 : 2;
    for (int i = 0; i < n_proj; ++i) {
        const int rc = validate_proj(projs[i], T, dtype);
        if (rc != LORDBA_OK) return rc;
    }
    if (T > 0) {
        // outputs must be pairwise disjoint and no input may lie in an output (n_proj is small:
        // 7 per layer, 224 per model)
        for (int i = 0; i < n_proj; ++i)
            for (int j = 0; j < n_proj; ++j) {
                if (i == j) continue;
                const size_t ni = ((size_t)(T - 1) * projs[i].ldy + projs[i].d_out) * e;
                const size_t nj = ((size_t)(T - 1) * projs[j].ldy + projs[j].d_out) * e;
                const size_t nx = ((size_t)(T - 1) * projs[i].ldx + projs[i].d_in) * e;
                if (j > i && overlaps(projs[i].y, ni, projs[j].y, nj)) return LORDBA_EINVAL;
                if (overlaps(projs[i].x, nx, projs[j].y, nj)) return LORDBA_EINVAL;
            }
    }
    if (T == 0 || n_proj == 0) return LORDBA_OK;
    return dispatch(projs, n_proj, T, nullptr, dtype, static_cast<cudaStream_t>(stream), true);
}

int lordba_adapter_forward_segments(const lordba_proj *segs, const int64_t *tokens, int n_seg, int dtype,
                                    void *stream)
{
    if (n_seg < 0 || (n_seg > 0 && (!segs || !tokens))) return LORDBA_EINVAL;
    const size_t e = (dtype == LORDBA_F32) ? 4 : 2;
    for (int i = 0; i < n_seg; ++i) {
        const int rc = validate_proj(segs[i], tokens[i], dtype);
        if (rc != LORDBA_OK) return rc;
    }
    // segments are simultaneous: outputs pairwise disjoint, no input inside an output
    for (int i = 0; i < n_seg; ++i)
        for (int j = 0; j < n_seg; ++j) {
            if (i == j || tokens[i] == 0 || tokens[j] == 0) continue;
            const size_t ni = ((size_t)(tokens[i] - 1) * segs[i].ldy + segs[i].d_out) * e;
            const size_t nj = ((size_t)(tokens[j] - 1) * segs[j].ldy + segs[j].d_out) * e;
            const size_t nx = ((size_t)(tokens[i] - 1) * segs[i].ldx + segs[i].d_in) * e;
            if (j > i && overlaps(segs[i].y, ni, segs[j].y, nj)) return LORDBA_EINVAL;
            if (overlaps(segs[i].x, nx, segs[j].y, nj)) return LORDBA_EINVAL;
        }
    if (n_seg == 0) return LORDBA_OK;
    return dispatch(segs, n_seg, 0, tokens, dtype, static_cast<cudaStream_t>(stream), true);
}

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
    const int rc2 = dispatch(&p, 1, T, nullptr, dtype, s, false);
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
