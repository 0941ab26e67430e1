// Helpers shared by the translation units of libhdet (not part of the C ABI).
#pragma once

#include <nvtx3/nvToolsExt.h>

namespace hdet {

// A named NVTX range around one C-ABI call, so that a timeline tool shows where the library's host time
// goes.  NVTX v3 is header-only: with no tool attached a range costs one predicted branch.
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// Stores the text that hdet_last_error(NULL) returns on the calling thread.
void set_handleless_error(const char* msg);

}  // namespace hdet
