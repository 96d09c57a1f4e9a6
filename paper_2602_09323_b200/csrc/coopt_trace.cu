// Host side of the trace build (see coopt_trace.cuh): where the caller's buffer is remembered.  Without
// -DCOOPT_TRACE this file is empty and the entry point does not exist.
#include "coopt_common.cuh"
#include "coopt_trace.cuh"

#ifdef COOPT_TRACE
namespace coopt {
namespace {
unsigned long long* g_trace_buffer = nullptr;
int g_plan_rotate = 0;
}
unsigned long long* trace_buffer() { return g_trace_buffer; }
int trace_plan_rotate() { return g_plan_rotate; }
}  // namespace coopt

// DEVICE buffer of kTraceMaxCtas * kTraceSlots uint64 (2 MiB), zeroed by the caller before a launch;
// NULL switches the stamps off.  Not thread-safe; a tool for one measuring process.
extern "C" int coopt_trace_set_buffer(void* device_buffer, size_t bytes) {
  if (device_buffer != nullptr && bytes < static_cast<size_t>(coopt::kTraceMaxCtas) * coopt::kTraceSlots * 8) return COOPT_ERR_WORKSPACE;
  coopt::g_trace_buffer = static_cast<unsigned long long*>(device_buffer);
  return COOPT_OK;
}

// CTA i of the decode kernel works through plan region (i + rotate) mod planned CTAs: tells apart what is slow
// because of its share of the plan from what is slow because of the SM it runs on.
extern "C" int coopt_trace_set_rotate(int rotate) {
  coopt::g_plan_rotate = rotate < 0 ? 0 : rotate;
  return COOPT_OK;
}
#endif
