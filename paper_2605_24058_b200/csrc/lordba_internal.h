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

// Cycles after which a bounded device-side wait gives up (about a second).  The test-hooks build
// (-DLORDBA_TEST_HOOKS, never the product library) cuts it to about a millisecond so that a test
// can watch a wait run out.
#ifdef LORDBA_TEST_HOOKS
constexpr long long kWaitLimitCycles = 2000000LL;
#else
constexpr long long kWaitLimitCycles = 1500000000LL;
#endif

// Test-hooks build only: index of the one pipeline item whose copy request the producer of the
// tensor-core kernels leaves out (-1 = none), so that the consumers' wait for it runs out with
// nothing in flight.  Always -1 in the product library.
int test_skip_item();

// Every kernel launch of the library goes through this counter.
void count_launch(int n = 1);

// Address of the device status word (resolved once per device).
int *device_status_word();

// ---- prepared launches ---------------------------------------------------------------------
// Every forward launcher describes its launches as records (kernel, grid, attributes, the
// kernel's argument blocks by value) and hands them to a sink.  The sink of a plain call
// launches each record at once; the sink of lordba_plan_init stores them in the caller's plan
// storage, and lordba_adapter_forward_planned replays them: the two paths launch the same
// kernels with the same arguments by construction.
struct LaunchRec {
    const void *func;
    uint32_t grid[3];
    uint32_t block;
    uint32_t smem;
    uint32_t cluster;      // CTAs per cluster (0 or 1: no cluster attribute)
    uint32_t pdl;          // 1: programmatic stream serialization allowed
    uint32_t n_args;       // 1 or 2 argument blocks
    uint32_t arg_bytes[2];
    uint32_t total_bytes;  // this record + its argument blocks in plan storage (multiple of 64)
    uint32_t cluster_z;    // 1: the cluster lies along grid z instead of grid x
};

struct LaunchSink {
    cudaStream_t stream = nullptr;
    bool immediate = true;   // launch now; otherwise append to buf (buf == nullptr: only count bytes)
    uint8_t *buf = nullptr;
    size_t cap = 0, used = 0;
    int count = 0;
    // arg1 may be null when rec.n_args == 1.  Returns a lordba_status.
    int emit(LaunchRec rec, const void *arg0, const void *arg1);
};

// Launch a stored record (args point into plan storage).
int launch_record(const LaunchRec &rec, const void *arg0, const void *arg1, cudaStream_t stream);

// A call holds at most this many projections (index arrays live on the stack).
constexpr int kMaxCallProjs = LORDBA_MAX_PROJS;

// Which projections of a call a launcher takes: those the selector maps to its own family.
struct FamilySelector {
    int dtype;
    int variant;       // the pinned family, or LORDBA_VARIANT_AUTO
    bool use_tc;       // AUTO decided for the tcgen05 kernel (or it is pinned)
    // LORDBA_VARIANT_FMA / _TC / _MMA for a projection with `rows` > 0 token rows; 0 for an empty one
    int family(const lordba_proj &p, int64_t rows) const;
};

// --- pack.cu ---------------------------------------------------------------
int launch_pack(const int8_t *signs, int64_t rows, int64_t cols, int role, uint32_t *packed,
                cudaStream_t stream);
int launch_widen_scales(const uint16_t *src, float *dst, int64_t n, cudaStream_t stream);
int launch_unpack(const uint32_t *packed, int64_t rows, int64_t cols, int role, int8_t *signs,
                  cudaStream_t stream);

// --- fit.cu ----------------------------------------------------------------
size_t fit_workspace_bytes(int64_t d_in, int64_t d_out, int r);
int launch_fit_scales(const float *target, int64_t ld, const uint32_t *pa, const uint32_t *pb, float *s_in, float *s_r,
                      float *s_out, int64_t d_in, int64_t d_out, int r, int sweeps, int axes, void *workspace,
                      cudaStream_t stream);

// --- forward_*.cu ------------------------------------------------------------
// Each launcher walks the n projections of a call (validated by the caller; tokens[i] = token
// rows of projection i, or T for all when tokens is null), takes those whose family is its own,
// and emits its launches into the sink.  *launches counts the launches of the call so far, over
// all families (the first launch of a call waits for the stream's previous kernel).
// batch_checked: the projections are known to be independent of one another, so the launches of
// this call may overlap each other; LORDBA_PROJ_OVERLAP on every projection lets the first
// launch overlap the previous call as well.
int launch_forward_fma(const lordba_proj *projs, const int64_t *tokens, int64_t T, int n, const FamilySelector &sel,
                       LaunchSink &sink);
bool tc_supported(const lordba_proj &p, int64_t T, int dtype);
int launch_forward_tc(const lordba_proj *projs, const int64_t *tokens, int64_t T, int n, const FamilySelector &sel,
                      LaunchSink &sink, bool batch_checked, int *launches);
bool mma_supported(const lordba_proj &p, int64_t T, int dtype);
int launch_forward_mma(const lordba_proj *projs, const int64_t *tokens, int64_t T, int n, const FamilySelector &sel,
                       LaunchSink &sink, bool batch_checked, int *launches);

inline int64_t rows_of(const int64_t *tokens, int64_t T, int i) { return tokens ? tokens[i] : T; }

}  // namespace lordba
