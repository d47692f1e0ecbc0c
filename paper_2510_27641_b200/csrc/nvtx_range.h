// NVTX range around a host-side entry point: shows up as a named span in a profiler's timeline
// and costs a null-pointer test when no tool is attached (NVTX v3 is header-only and loads the
// tool's library on demand).
#pragma once
#include <nvtx3/nvToolsExt.h>

namespace specattn {
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};
}  // namespace specattn
