// Internal declarations shared by the translation units of liblordba.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "lordba.h"

namespace lordba {

constexpr int kMaxRank = 64;

// Device status codes written by bounded waits (0 = none).
enum DeviceCode : int {
    kDevOk = 0,
    kDevTmaWaitTimeout = 1,
    kDevMmaWaitTimeout = 2,
    kDevClusterWaitTimeout = 3,
    kDevEpilogueWaitTimeout = 4,
};

// Every kernel launch of the library goes through this counter.
void count_launch(int n = 1);

// Address of the device status word (resolved once per device).
int *device_status_word();

// --- pack.cu ---------------------------------------------------------------
int launch_pack(const int8_t *signs, int64_t rows, int64_t cols, int role, uint32_t *packed,
                cudaStream_t stream);
int launch_widen_scales(const uint16_t *src, float *dst, int64_t n, cudaStream_t stream);
int launch_unpack(const uint32_t *packed, int64_t rows, int64_t cols, int role, int8_t *signs,
                  cudaStream_t stream);

// --- forward_fma.cu ----------------------------------------------------------
// n projections (validated by the caller), same T and dtype.  Any shape.
// tokens[i]: token rows of projection i (entries may differ; zero entries are skipped).
int launch_forward_fma(const lordba_proj *projs, const int64_t *tokens, int n, int dtype, cudaStream_t stream);

// --- forward_tc.cu -----------------------------------------------------------
// True when the tcgen05/TMA kernel can take this projection (bf16, 16-byte
// aligned rows, rank a multiple of 8).
bool tc_supported(const lordba_proj &p, int64_t T, int dtype);
int launch_forward_tc(const lordba_proj *projs, int n, int64_t T, int dtype, cudaStream_t stream,
                      bool batch_checked);

// --- forward_mma.cu ----------------------------------------------------------
// True when the register-streaming mma.sync kernel can take this projection
// (bf16, 16-byte aligned rows, widths and rank multiples of 8).
bool mma_supported(const lordba_proj &p, int64_t T, int dtype);
// batch_checked: the projections are known to be independent of one another, so the launches of
// this call may overlap each other; LORDBA_PROJ_OVERLAP on every projection lets the first
// launch overlap the previous call as well.
int launch_forward_mma(const lordba_proj *projs, const int64_t *tokens, int n, int dtype, cudaStream_t stream,
                       bool batch_checked);

}  // namespace lordba
