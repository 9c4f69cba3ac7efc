#include "common.cuh"

#include <atomic>

namespace tv {

char* error_buffer() {
  static thread_local char buf[512] = {0};
  return buf;
}

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(error_buffer(), 512, fmt, ap);
  va_end(ap);
  return code;
}

static std::atomic<unsigned long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

}  // namespace tv

extern "C" const char* tv_last_error(void) { return tv::error_buffer(); }
extern "C" int tv_version(void) { return 100; }
extern "C" unsigned long long tv_launch_count(void) { return tv::g_launches.load(std::memory_order_relaxed); }
