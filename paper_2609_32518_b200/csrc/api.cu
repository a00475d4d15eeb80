// Status text and the launch counter of the C ABI.
#include "attn_sched.h"
#include "common.h"

namespace unstep {
std::atomic<int64_t> g_launches{0};
}

extern "C" const char* unstep_strerror(int code) {
  switch (code) {
    case UNSTEP_OK: return "ok";
    case UNSTEP_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, bad size or window)";
    case UNSTEP_ERR_UNSUPPORTED: return "unsupported (head_dim must be 128, device must be sm_100)";
    case UNSTEP_ERR_CUDA: return "a CUDA call failed";
    case UNSTEP_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case UNSTEP_ERR_TOO_LARGE: return "too large for the fixed scratch of the no-allocation entry point";
    case UNSTEP_ERR_BOUNDS: return "checking build: a kernel tried to store outside its buffer (the store was skipped)";
    default: return "unknown status";
  }
}

extern "C" int64_t unstep_launch_count(void) { return unstep::g_launches.load(); }


// The work split of an attention launch, listed on the host with the same code the kernel's
// roles run on the device.
extern "C" int unstep_window_attn_plan(const unstep_shape_t* shape, int32_t sink_frames,
                                       const int32_t* start_frame, int32_t recent_frames,
                                       int32_t sink_attend, int32_t max_workers, int32_t* segs,
                                       int32_t max_segs, int32_t* n_segs) {
  using namespace unstep;
  int rc = check_attn_args(shape, start_frame, recent_frames, sink_frames, sink_attend);
  if (rc != UNSTEP_OK) return rc;
  if (max_workers < 1 || max_workers > 65536 || n_segs == nullptr || max_segs < 0 ||
      (segs == nullptr && max_segs > 0))
    return UNSTEP_ERR_INVALID_ARG;
  AttnParams p;
  plan_shape(p, shape, sink_frames);
  const int nb = shape->batch < kMaxStreamsPerLaunch ? shape->batch : kMaxStreamsPerLaunch;
  rc = plan_launch(p, shape, start_frame, nb, recent_frames, sink_frames, sink_attend, max_workers);
  if (rc != UNSTEP_OK) return rc;
  int64_t n = 0;
  for (int w = 0; w < p.n_workers; ++w) {
    Sched sched(p, w);
    Seg s;
    while (sched.next(s)) {
      if (n < max_segs) {
        const bool whole = s.t0 == 0 && s.t1 == s.tiles;
        int32_t* o = segs + 10 * n;
        o[0] = w;
        o[1] = s.b;
        o[2] = s.h;
        o[3] = s.qp;
        o[4] = s.nq;
        o[5] = s.t0;
        o[6] = s.t1;
        o[7] = s.tiles;
        o[8] = whole ? 1 : last_part_worker(p, s) - first_part_worker(p, s) + 1;
        o[9] = whole ? -1 : part_slot(p, w, s.item_step0);
      }
      ++n;
    }
  }
  if (n > INT32_MAX) return UNSTEP_ERR_INVALID_ARG;
  *n_segs = static_cast<int32_t>(n);
  return UNSTEP_OK;
}
