// Index checks of the "bounds" build and the bits of the device error word.
#pragma once

#include <stdint.h>

namespace slaq {

// Bits of the device error word (slaq_handle::err_word).  kErrWindow and kErrInput are set by every build; the
// others only by the "bounds" build (-DSLAQ_DEBUG_BOUNDS), in which every index into a ring, the
// packed pool, a shared-memory slice, the gain table, a candidate segment, a histogram or a per-job
// array is compared with its extent first: a bad index sets its bit and the access is skipped (a
// skipped read gives zero), nothing traps.  slaq_schedule reports a non-zero word as SLAQ_E_CUDA.
enum : int32_t {
    kErrWindow = 1,     // a job's stored count exceeds its ring or the longest window the launch was sized for
    kErrStorage = 2,    // a position outside a job's ring, or a ring outside the pools
    kErrShared = 4,     // an offset outside a warp's shared-memory slice or the weight table
    kErrGain = 8,       // an entry outside the gain table
    kErrSegment = 16,   // a candidate segment that does not lie inside its row
    kErrBin = 32,       // a histogram bin or window-length bucket out of range
    kErrJob = 64,       // a job id or work-list position out of range
    kErrInput = 128     // set by every build: device-side input of slaq_append_losses_device that had to be skipped
};

#ifdef SLAQ_DEBUG_BOUNDS
__device__ __forceinline__ bool index_ok(long long i, long long n, int32_t bit, int32_t* err_word) {
    if (i >= 0 && i < n) return true;
    if (err_word) atomicOr(err_word, bit);
    return false;
}
#else
__device__ __forceinline__ bool index_ok(long long, long long, int32_t, int32_t*) { return true; }
#endif

}  // namespace slaq
