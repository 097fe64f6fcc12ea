// Launch accounting and optional per-kernel CUDA-event timing (diagnostics; off by default).
// Not thread-safe: meant for a single-threaded benchmark driver.
#include <string.h>

#include "cvlc_common.cuh"

namespace cvlc {

namespace {
const char* const kKernelNames[kNumKernelIds] = {
    "k_zero_words", "k_hist", "k_plan", "k_encode_init", "k_select", "k_select_lookback", "k_sort_hist", "k_sort_scan", "k_sort_pass", "k_pack",
    "k_decode_prepare", "k_fill_zero", "k_decode", "k_selftest"};

unsigned long long g_launches[kNumKernelIds] = {};
int g_prof_kernel = -1;
uint32_t g_prof_capacity = 0, g_prof_count = 0;
cudaEvent_t* g_prof_events = nullptr;  // 2 per timed launch
}  // namespace

void launch_begin(int id, cudaStream_t st) {
  g_launches[id] += 1;
  if (id == g_prof_kernel && g_prof_count < g_prof_capacity) cudaEventRecord(g_prof_events[2 * g_prof_count], st);
}

void launch_end(int id, cudaStream_t st) {
  if (id == g_prof_kernel && g_prof_count < g_prof_capacity) {
    cudaEventRecord(g_prof_events[2 * g_prof_count + 1], st);
    g_prof_count += 1;
  }
}

}  // namespace cvlc

using namespace cvlc;

extern "C" {

unsigned long long cvlc_launch_count(const char* kernel_name) {
  unsigned long long total = 0;
  for (int i = 0; i < kNumKernelIds; ++i)
    if (!kernel_name || !kernel_name[0] || strcmp(kernel_name, kKernelNames[i]) == 0) total += g_launches[i];
  return total;
}

int cvlc_profile_select(const char* kernel_name, uint32_t max_launches) {
  if (g_prof_events) {
    for (uint32_t i = 0; i < 2 * g_prof_capacity; ++i) cudaEventDestroy(g_prof_events[i]);
    delete[] g_prof_events;
    g_prof_events = nullptr;
  }
  g_prof_kernel = -1;
  g_prof_capacity = g_prof_count = 0;
  if (!kernel_name || !kernel_name[0] || max_launches == 0) return CVLC_OK;
  int id = -1;
  for (int i = 0; i < kNumKernelIds; ++i)
    if (strcmp(kernel_name, kKernelNames[i]) == 0) id = i;
  if (id < 0) return CVLC_ERR_INVALID_ARG;
  g_prof_events = new cudaEvent_t[2 * (size_t)max_launches];
  for (uint32_t i = 0; i < 2 * max_launches; ++i)
    if (cudaEventCreate(&g_prof_events[i]) != cudaSuccess) return CVLC_ERR_CUDA;
  g_prof_capacity = max_launches;
  g_prof_kernel = id;
  return CVLC_OK;
}

int cvlc_profile_reset(void) {
  g_prof_count = 0;
  return CVLC_OK;
}

int cvlc_profile_read(uint32_t* launches, double* total_ms) {
  if (!launches || !total_ms) return CVLC_ERR_INVALID_ARG;
  *launches = 0;
  *total_ms = 0.0;
  if (cudaDeviceSynchronize() != cudaSuccess) return CVLC_ERR_CUDA;
  for (uint32_t i = 0; i < g_prof_count; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, g_prof_events[2 * i], g_prof_events[2 * i + 1]) != cudaSuccess) return CVLC_ERR_CUDA;
    *total_ms += (double)ms;
  }
  *launches = g_prof_count;
  return CVLC_OK;
}

}  // extern "C"
