// Bit-packing of the +-1 carriers ("bit-packed {B1,B2}", Section 3.3).
//
// Both roles are a flat ballot: a warp reads 32 consecutive int8 signs and one
// lane writes the word.  Role 1 (B carrier) is the flat row-major stream
// itself; role 0 (A carrier) is the same per row, each row padded to whole
// words.  sign(0) = +1: an entry packs as bit 0 only when it is negative.
#include "lordba_internal.h"

namespace lordba {
namespace {

constexpr int kPackThreads = 256;

// rows x cols int8 -> rows x ceil(cols/32) words; role 1 calls it with rows = 1
// and cols = d_out * r.
__global__ void __launch_bounds__(kPackThreads)
pack_rows_kernel(const int8_t *__restrict__ signs, int64_t rows, int64_t cols, int64_t words_per_row,
                 uint32_t *__restrict__ packed)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (kPackThreads / 32) + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * (kPackThreads / 32);
    const int64_t total = rows * words_per_row;
    for (int64_t w = warp; w < total; w += n_warps) {
        const int64_t row = w / words_per_row;
        const int64_t col = (w - row * words_per_row) * 32 + lane;
        bool plus = false;
        if (col < cols) plus = signs[row * cols + col] >= 0;
        const uint32_t word = __ballot_sync(0xffffffffu, plus);
        if (lane == 0) packed[w] = word;
    }
}

__global__ void __launch_bounds__(kPackThreads)
unpack_rows_kernel(const uint32_t *__restrict__ packed, int64_t rows, int64_t cols,
                   int64_t words_per_row, int8_t *__restrict__ signs)
{
    const int64_t total = rows * cols;
    const int64_t stride = (int64_t)gridDim.x * kPackThreads;
    for (int64_t e = (int64_t)blockIdx.x * kPackThreads + threadIdx.x; e < total; e += stride) {
        const int64_t row = e / cols;
        const int64_t col = e - row * cols;
        const uint32_t word = packed[row * words_per_row + (col >> 5)];
        signs[e] = ((word >> (col & 31)) & 1u) ? (int8_t)1 : (int8_t)-1;
    }
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
    const int64_t wpr = (pcols + 31) / 32;
    if (prow * wpr == 0) return LORDBA_OK;
    pack_rows_kernel<<<grid_for(prow * wpr, kPackThreads / 32), kPackThreads, 0, stream>>>(
        signs, prow, pcols, wpr, packed);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LORDBA_OK : LORDBA_ECUDA;
}

int launch_unpack(const uint32_t *packed, int64_t rows, int64_t cols, int role, int8_t *signs,
                  cudaStream_t stream)
{
    int64_t prow = rows, pcols = cols;
    if (role == 1) { prow = 1; pcols = rows * cols; }
    const int64_t wpr = (pcols + 31) / 32;
    if (prow * pcols == 0) return LORDBA_OK;
    unpack_rows_kernel<<<grid_for(prow * pcols, kPackThreads), kPackThreads, 0, stream>>>(
        packed, prow, pcols, wpr, signs);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LORDBA_OK : LORDBA_ECUDA;
}

}  // namespace lordba
