// Index checks of the debug build (-DSP_DEBUG_CHECKS).  A checked access whose index is out of
// range is skipped and recorded - the first offender with its kernel-specific code, block,
// thread, index and limit, plus a count - instead of faulting; nothing traps.  In the release
// build SP_IN_RANGE is the constant true and the checks vanish.  Every translation unit that
// uses the macro keeps its own record; sp_debug_status (api.cu) collects them through the
// readers registered here.
#pragma once

#include <cuda_runtime.h>

namespace sp {

struct DebugRecord {
    unsigned int count;  // violations seen
    int code;            // which check (kDbg*)
    int block, thread;
    long long index, limit;
};
typedef cudaError_t (*DebugReader)(DebugRecord *out, bool clear);
void register_debug_reader(DebugReader reader);  // api.cu

// codes of the checked accesses
constexpr int kDbgCalibPartial = 1;   // calib_accumulate_kernel: partial-sum row
constexpr int kDbgFactorPairs = 2;    // finalize_kernel: tile-ordered factor copy
constexpr int kDbgNmRow = 3;          // select_nm_stream_kernel: row of a job
constexpr int kDbgNmColumn = 4;       // ... column within the leading dimension
constexpr int kDbgEwmaColumn = 5;     // ewma_pair_scan_kernel: column of a pruned chunk
constexpr int kDbgEwmaMask = 6;       // ... mask half-word of a row
constexpr int kDbgWalkMask = 7;       // literal_walk: mask word of a row

#ifdef SP_DEBUG_CHECKS
static __device__ DebugRecord g_debug_record;

__device__ __forceinline__ bool debug_in_range(long long index, long long limit, int code) {
    if (index >= 0 && index < limit) return true;
    if (atomicAdd(&g_debug_record.count, 1u) == 0u) {
        g_debug_record.code = code;
        g_debug_record.block = static_cast<int>(blockIdx.x + gridDim.x * blockIdx.y);
        g_debug_record.thread = static_cast<int>(threadIdx.x);
        g_debug_record.index = index;
        g_debug_record.limit = limit;
    }
    return false;
}

static cudaError_t debug_read_this_unit(DebugRecord *out, bool clear) {
    cudaError_t e = cudaMemcpyFromSymbol(out, g_debug_record, sizeof(DebugRecord));
    if (e == cudaSuccess && clear) {
        const DebugRecord zero = {};
        e = cudaMemcpyToSymbol(g_debug_record, &zero, sizeof(DebugRecord));
    }
    return e;
}
namespace {
struct DebugRegistration {
    DebugRegistration() { register_debug_reader(debug_read_this_unit); }
};
const DebugRegistration g_debug_registration;
}  // namespace

#define SP_IN_RANGE(index, limit, code) \
    ::sp::debug_in_range(static_cast<long long>(index), static_cast<long long>(limit), (code))
#else
#define SP_IN_RANGE(index, limit, code) (true)
#endif

}  // namespace sp
