// Bit-packing of the +-1 carriers ("bit-packed {B1,B2}", Section 3.3).
//
// A warp reads 32 consecutive int8 signs of one row and one lane writes the
// ballot.  Role 1 (B carrier, d_out x r) is the flat row-major bit stream.
// Role 0 (A carrier, r x d_in) is block-major: for every block of 64 columns,
// r consecutive 64-bit groups (two words each, low word first), one per row.
// sign(0) = +1: an entry packs as bit 0 only when it is negative.
#include <cuda_fp16.h>

#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kPackThreads = 256;

// Word w of the packed array -> (row, first column) of the 32 signs it holds.
__device__ __forceinline__ void word_to_source(int64_t w, int64_t rows, int role, int64_t &row, int64_t &col0)
{
    if (role == 0) {
        const int64_t block = w / (rows * 2);
        const int64_t rem = w - block * rows * 2;
        row = rem >> 1;
        col0 = block * 64 + (rem & 1) * 32;
    } else {            // flat stream: the caller passes rows = 1, cols = d_out * r
        row = 0;
        col0 = w * 32;
    }
}

__global__ void __launch_bounds__(kPackThreads)
pack_kernel(const int8_t *__restrict__ signs, int64_t rows, int64_t cols, int role, int64_t total_words,
            uint32_t *__restrict__ packed)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (kPackThreads / 32) + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * (kPackThreads / 32);
    for (int64_t w = warp; w < total_words; w += n_warps) {
        int64_t row, col0;
        word_to_source(w, rows, role, row, col0);
        const int64_t col = col0 + lane;
        bool plus = false;
        if (col < cols) plus = signs[row * cols + col] >= 0;
        const uint32_t word = __ballot_sync(0xffffffffu, plus);
        if (lane == 0) packed[w] = word;
    }
}

__global__ void __launch_bounds__(kPackThreads)
unpack_kernel(const uint32_t *__restrict__ packed, int64_t rows, int64_t cols, int role,
              int8_t *__restrict__ signs)
{
    const int64_t total = rows * cols;
    const int64_t stride = (int64_t)gridDim.x * kPackThreads;
    for (int64_t e = (int64_t)blockIdx.x * kPackThreads + threadIdx.x; e < total; e += stride) {
        const int64_t row = e / cols;
        const int64_t col = e - row * cols;
        const int64_t w = (role == 0) ? ((col >> 6) * rows + row) * 2 + ((col & 63) >> 5) : (e >> 5);
        const int bit = (role == 0) ? (int)(col & 31) : (int)(e & 31);
        signs[e] = ((packed[w] >> bit) & 1u) ? (int8_t)1 : (int8_t)-1;
    }
}

// Exported adapters store their scales as IEEE halves; the forward kernels take float32.
__global__ void __launch_bounds__(kPackThreads)
widen_scales_kernel(const __half *__restrict__ src, float *__restrict__ dst, int64_t n)
{
    const int64_t stride = (int64_t)gridDim.x * kPackThreads;
    for (int64_t e = (int64_t)blockIdx.x * kPackThreads + threadIdx.x; e < n; e += stride)
        dst[e] = __half2float(src[e]);
}

int grid_for(int64_t work_items, int per_block)
{
    int64_t blocks = (work_items + per_block - 1) / per_block;
    if (blocks < 1) blocks = 1;
    if (blocks > 148 * 16) blocks = 148 * 16;
    return (int)blocks;
}

}  // namespace

int launch_pack(const int8_t *signs, int64_t rows, int64_t cols, int role, uint32_t *packed,
                cudaStream_t stream)
{
    int64_t prow = rows, pcols = cols;
    if (role == 1) { prow = 1; pcols = rows * cols; }
    const int64_t words = (role == 0) ? ((cols + 63) / 64) * rows * 2 : (pcols + 31) / 32;
    if (words == 0) return LORDBA_OK;
    pack_kernel<<<grid_for(words, kPackThreads / 32), kPackThreads, 0, stream>>>(signs, prow, pcols, role,
                                                                                words, packed);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LORDBA_OK : LORDBA_ECUDA;
}

int launch_widen_scales(const uint16_t *src, float *dst, int64_t n, cudaStream_t stream)
{
    if (n == 0) return LORDBA_OK;
    widen_scales_kernel<<<grid_for(n, kPackThreads), kPackThreads, 0, stream>>>(
        reinterpret_cast<const __half *>(src), dst, n);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LORDBA_OK : LORDBA_ECUDA;
}

int launch_unpack(const uint32_t *packed, int64_t rows, int64_t cols, int role, int8_t *signs,
                  cudaStream_t stream)
{
    int64_t prow = rows, pcols = cols;
    if (role == 1) { prow = 1; pcols = rows * cols; }
    if (prow * pcols == 0) return LORDBA_OK;
    unpack_kernel<<<grid_for(prow * pcols, kPackThreads), kPackThreads, 0, stream>>>(packed, prow, pcols,
                                                                                     role, signs);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LORDBA_OK : LORDBA_ECUDA;
}

}  // namespace lordba
