// Host-side helpers shared by the entry points: argument checks and the launch counter.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "unstep.h"

namespace unstep {

constexpr int kHeadDim = 128;
constexpr int kPairs = 64;
constexpr int kMaxStreamsPerLaunch = 32;  // per-stream host scalars travel as kernel parameters

extern std::atomic<int64_t> g_launches;

// Device address of the status word on the current device (null if it cannot be found).
int* status_word();

// A checking build (-DUNSTEP_CHECK) tests every global store of the kernels against the extent of
// the buffer it belongs to; a store outside is skipped and recorded in the status word (no trap),
// so that a wrong index shows up as UNSTEP_ERR_BOUNDS instead of silent corruption.  This stands
// in for a memory checker where none can be run.  In a normal build the macro is the plain store.
#ifdef UNSTEP_CHECK
#define UNSTEP_STORE(base, idx, extent, value, status)                                  \
  do {                                                                                  \
    const long long idx_ = static_cast<long long>(idx);                                 \
    if (idx_ >= 0 && idx_ < static_cast<long long>(extent)) (base)[idx_] = (value);     \
    else atomicExch((status), static_cast<int>(UNSTEP_ERR_BOUNDS));                     \
  } while (0)
#else
#define UNSTEP_STORE(base, idx, extent, value, status) ((base)[idx] = (value))
#endif

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shape checks common to every call.  `need_ring` also checks batch/heads/ring_frames.
inline int check_shape(const unstep_shape_t* s, bool need_ring) {
  if (s == nullptr) return UNSTEP_ERR_INVALID_ARG;
  if (s->head_dim != kHeadDim) return s->head_dim > 0 ? UNSTEP_ERR_UNSUPPORTED : UNSTEP_ERR_INVALID_ARG;
  if (s->chunk_frames <= 0 || s->grid_h <= 0 || s->grid_w <= 0) return UNSTEP_ERR_INVALID_ARG;
  if (s->band_t <= 0 || s->band_h <= 0 || s->band_w <= 0) return UNSTEP_ERR_INVALID_ARG;
  if ((s->band_t | s->band_h | s->band_w) & 1) return UNSTEP_ERR_INVALID_ARG;
  if (s->band_t + s->band_h + s->band_w != s->head_dim) return UNSTEP_ERR_INVALID_ARG;
  if (!(s->rope_base > 0.0)) return UNSTEP_ERR_INVALID_ARG;
  const int64_t T = static_cast<int64_t>(s->grid_h) * s->grid_w;
  const int64_t L = T * s->chunk_frames;
  if (T > (1 << 24) || L > (1 << 26)) return UNSTEP_ERR_INVALID_ARG;
  if (need_ring) {
    if (s->batch <= 0 || s->heads <= 0 || s->ring_frames <= 0) return UNSTEP_ERR_INVALID_ARG;
    if (s->ring_frames < s->chunk_frames) return UNSTEP_ERR_INVALID_ARG;
    if (s->heads > 4096 || s->batch > (1 << 20)) return UNSTEP_ERR_INVALID_ARG;
    // element offsets inside one stream's ring must fit comfortably in 63 bits / TMA strides in 40
    const int64_t ring_elems = static_cast<int64_t>(s->ring_frames) * T * s->heads * kHeadDim;
    if (ring_elems > (int64_t(1) << 38)) return UNSTEP_ERR_INVALID_ARG;
  }
  return UNSTEP_OK;
}

// The device the call will run on must be sm_100.
inline int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return UNSTEP_ERR_CUDA;
  static thread_local int cached_dev = -1, cached_major = 0;
  if (cached_dev != dev) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return UNSTEP_ERR_CUDA;
    cached_dev = dev;
    cached_major = major;
  }
  return cached_major == 10 ? UNSTEP_OK : UNSTEP_ERR_UNSUPPORTED;
}

}  // namespace unstep
