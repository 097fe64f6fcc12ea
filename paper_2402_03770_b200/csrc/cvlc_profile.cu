// Launch accounting and optional per-kernel CUDA-event timing (diagnostics; off by default).
// Not thread-safe: meant for a single-threaded benchmark driver.
#include <string.h>

#include "cvlc_common.cuh"

namespace cvlc {

namespace {
const char* const kKernelNames[kNumKernelIds] = {
    "k_zero_words", "k_hist", "k_plan_fit", "k_plan_tune", "k_plan_finish", "k_encode_init", "k_select", "k_select_lookback", "k_sort_hist",
    "k_sort_scan", "k_sort_pass", "k_pack", "k_decode_prepare", "k_fill_zero", "k_prefetch_l2", "k_decode", "k_noalloc_publish_status",
    "k_selftest", "k_hist_check", "k_apply", "k_plan_literal", "k_ec_accumulate", "k_pack_unframed", "k_decode_unframed"};

unsigned long long g_launches[kNumKernelIds] = {};
int g_prof_kernel = -1;          // kernel id being timed; kNumKernelIds = every kernel; -1 = off
uint32_t g_prof_capacity = 0, g_prof_count = 0;
cudaEvent_t* g_prof_events = nullptr;  // 2 per timed launch
int* g_prof_ids = nullptr;             // kernel id of every timed launch
}  // namespace

static inline bool prof_wants(int id) {
  return (g_prof_kernel == id || g_prof_kernel == kNumKernelIds) && g_prof_count < g_prof_capacity;
}

void launch_begin(int id, cudaStream_t st) {
  g_launches[id] += 1;
  if (prof_wants(id)) cudaEventRecord(g_prof_events[2 * g_prof_count], st);
}

void launch_end(int id, cudaStream_t st) {
  if (prof_wants(id)) {
    cudaEventRecord(g_prof_events[2 * g_prof_count + 1], st);
    g_prof_ids[g_prof_count] = id;
    g_prof_count += 1;
  }
}

}  // namespace cvlc

using namespace cvlc;

static int kernel_id_of(const char* name) {
  for (int i = 0; i < kNumKernelIds; ++i)
    if (strcmp(name, kKernelNames[i]) == 0) return i;
  return -1;
}

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
    delete[] g_prof_ids;
    g_prof_events = nullptr;
    g_prof_ids = nullptr;
  }
  g_prof_kernel = -1;
  g_prof_capacity = g_prof_count = 0;
  if (!kernel_name || !kernel_name[0] || max_launches == 0) return CVLC_OK;
  const int id = (strcmp(kernel_name, "*") == 0) ? (int)kNumKernelIds : kernel_id_of(kernel_name);
  if (id < 0) return CVLC_ERR_INVALID_ARG;
  g_prof_events = new cudaEvent_t[2 * (size_t)max_launches];
  g_prof_ids = new int[max_launches];
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

int cvlc_profile_read(const char* kernel_name, uint32_t* launches, double* total_ms) {
  if (!launches || !total_ms) return CVLC_ERR_INVALID_ARG;
  *launches = 0;
  *total_ms = 0.0;
  const int want = (!kernel_name || !kernel_name[0] || strcmp(kernel_name, "*") == 0) ? -1 : kernel_id_of(kernel_name);
  if (kernel_name && kernel_name[0] && strcmp(kernel_name, "*") != 0 && want < 0) return CVLC_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return CVLC_ERR_CUDA;
  for (uint32_t i = 0; i < g_prof_count; ++i) {
    if (want >= 0 && g_prof_ids[i] != want) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, g_prof_events[2 * i], g_prof_events[2 * i + 1]) != cudaSuccess) return CVLC_ERR_CUDA;
    *total_ms += (double)ms;
    *launches += 1;
  }
  return CVLC_OK;
}

}  // extern "C"
