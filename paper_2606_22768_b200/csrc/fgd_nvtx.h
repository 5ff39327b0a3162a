// NVTX range around each C-ABI entry point, so that a timeline profiler shows the library's calls
// by name.  NVTX v3 is header-only: without a profiler attached a push / pop is a load and a
// branch.
#ifndef FGD_NVTX_H_
#define FGD_NVTX_H_

#include <nvtx3/nvToolsExt.h>

namespace fgd {
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};
}  // namespace fgd
#define FGD_NVTX_RANGE(name) ::fgd::NvtxRange fgd_nvtx_range_(name)
#endif
