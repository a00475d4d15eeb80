// Status text and the launch counter of the C ABI.
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
    default: return "unknown status";
  }
}

extern "C" int64_t unstep_launch_count(void) { return unstep::g_launches.load(); }
