// oilbird_query_static: the single-request query for callers that must not allocate.
//
// Some hosts of this library own every byte of device memory themselves: a serving
// engine that reserved all of HBM for its KV cache and weights at start-up, or a
// real-time loop whose policy forbids driver allocations once it is running (an
// allocation there can fail, stall the stream or fragment the reservation).  Such a
// caller keeps the pool's arrays inside its own reservation and cannot let the library
// cudaMalloc the candidate lists that the scan hands to the merge.  For them the scratch
// lives in a fixed array that is part of the library image; the call below runs the same
// CUDA-core scan and the same merge/gather kernels as oilbird_pool_query on it.
//
// The array is reserved on every GPU that loads the library, until the process exits.
// All calls on a device share it and it keeps the previous call's contents: every word a
// call reads is rewritten by that call first (candidate lists, query-valid flags) and the
// counters are cleared at the start of each call.  Two calls that overlap on one GPU
// (different streams, or different threads) race on it.
#include <stdio.h>

#include "internal.h"

namespace oilbird {

// Limits of the static variant: at most 2 queries per call, k <= 128, and up to
// kStaticMaxLists candidate lists (the scan launches two CTAs per SM, so this covers
// GPUs of up to 256 SMs).  512 * 2 * 128 * 8 bytes = 1 MiB, plus flags and counters.
constexpr int kStaticMaxNq = OILBIRD_STATIC_MAX_NQ;
constexpr int kStaticMaxLists = 512;
constexpr size_t kStaticListBytes = (size_t)kStaticMaxLists * kStaticMaxNq * OILBIRD_MAX_K * 8;
constexpr size_t kStaticFlagBytes = 256;     // q_valid[2], padded
constexpr size_t kStaticBytes = kStaticListBytes + kStaticFlagBytes + 256 /* DeviceStats */;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// In host code the name above is only a stand-in for the symbol; the device address has
// to be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
static unsigned char* g_scratch_ptr[kMaxDevices];
static int g_num_sms[kMaxDevices];
static char g_static_err[256] = "";

static int static_setup(int device) {
  if (g_scratch_ptr[device]) return OILBIRD_OK;
  if (preload_all_kernels() != cudaSuccess) {      // first use on this device
    snprintf(g_static_err, sizeof g_static_err, "loading the library's kernels failed");
    return OILBIRD_ECUDA;
  }
  void* p = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
  if (e != cudaSuccess || !p) {
    snprintf(g_static_err, sizeof g_static_err, "cudaGetSymbolAddress(static scratch): %s",
             cudaGetErrorString(e));
    return OILBIRD_ECUDA;
  }
  int sms = 0;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  if (e != cudaSuccess || sms < 1) {
    snprintf(g_static_err, sizeof g_static_err, "cudaDeviceGetAttribute(SM count): %s",
             cudaGetErrorString(e));
    return OILBIRD_ECUDA;
  }
  g_num_sms[device] = sms;
  g_scratch_ptr[device] = (unsigned char*)p;
  return OILBIRD_OK;
}

}  // namespace oilbird

using namespace oilbird;

extern "C" {

const char* oilbird_query_static_error(void) { return g_static_err; }

int oilbird_query_static(const oilbird_static_pool* sp, const void* q_bf16, int32_t nq,
                         const oilbird_query_params* pr, const oilbird_query_out* out,
                         void* cuda_stream) {
  g_static_err[0] = 0;
  if (!sp || !q_bf16 || !pr || !out || !out->idx || !out->score || !out->fired ||
      !out->cont_len || !out->cont_tok ||
      (sp->n_rows > 0 && (!sp->keys || !sp->tokens || !sp->trace_id || !sp->trace_end))) {
    snprintf(g_static_err, sizeof g_static_err, "null argument");
    return OILBIRD_EINVAL;
  }
  if (sp->device < 0 || sp->device >= kMaxDevices) {
    snprintf(g_static_err, sizeof g_static_err, "device ordinal %d out of range", sp->device);
    return OILBIRD_EINVAL;
  }
  if (nq < 1 || nq > kStaticMaxNq) {
    snprintf(g_static_err, sizeof g_static_err,
             "nq=%d exceeds the static scratch (at most %d queries per call)", nq, kStaticMaxNq);
    return OILBIRD_EINVAL;
  }
  if (pr->k < 1 || pr->k > OILBIRD_MAX_K) {
    snprintf(g_static_err, sizeof g_static_err,
             "k=%d exceeds the static scratch (at most %d neighbours)", pr->k, OILBIRD_MAX_K);
    return OILBIRD_EINVAL;
  }
  if (sp->d < 8 || sp->d > 16384 || sp->d % 8 != 0 || sp->n_rows < 0 ||
      sp->n_rows > 2147483000LL) {
    snprintf(g_static_err, sizeof g_static_err, "pool geometry out of range (d=%d, rows=%lld)",
             sp->d, (long long)sp->n_rows);
    return OILBIRD_EINVAL;
  }
  GatherParams gp;
  if (check_query_params(nq, kStaticMaxNq, OILBIRD_MAX_K, pr, &gp) != OILBIRD_OK) {
    snprintf(g_static_err, sizeof g_static_err, "query parameter out of range");
    return OILBIRD_EINVAL;
  }
  if (pr->exclude_tag || pr->path == OILBIRD_PATH_TENSOR || pr->path == OILBIRD_PATH_MMA) {
    snprintf(g_static_err, sizeof g_static_err,
             "the static variant has no exclusion tags and only the CUDA-core scan");
    return OILBIRD_EINVAL;
  }
  // the kernels read keys and queries with 16-byte loads and the integer arrays word by word
  const uintptr_t a16 = (uintptr_t)q_bf16 | (sp->n_rows > 0 ? (uintptr_t)sp->keys : 0);
  const uintptr_t a4 = (uintptr_t)out->idx | (uintptr_t)out->score | (uintptr_t)out->fired |
                       (uintptr_t)out->cont_len | (uintptr_t)out->cont_tok |
                       (sp->n_rows > 0 ? (uintptr_t)sp->tokens | (uintptr_t)sp->trace_id |
                                             (uintptr_t)sp->trace_end : 0);
  if ((a16 & 15) || (a4 & 3)) {
    snprintf(g_static_err, sizeof g_static_err,
             "misaligned pointer (keys and q: 16 bytes; integer and score arrays: 4 bytes)");
    return OILBIRD_EINVAL;
  }
  cudaError_t e = cudaSetDevice(sp->device);
  if (e != cudaSuccess) {
    snprintf(g_static_err, sizeof g_static_err, "cudaSetDevice: %s", cudaGetErrorString(e));
    return OILBIRD_ECUDA;
  }
  int rc = static_setup(sp->device);
  if (rc) return rc;
  unsigned char* base = g_scratch_ptr[sp->device];
  unsigned long long* partial = (unsigned long long*)base;
  int32_t* q_valid = (int32_t*)(base + kStaticListBytes);
  DeviceStats* stats = (DeviceStats*)(base + kStaticListBytes + kStaticFlagBytes);
  cudaStream_t st = (cudaStream_t)cuda_stream;

  PoolView pv;
  pv.keys = (const uint16_t*)sp->keys; pv.tok = sp->tokens; pv.trace_id = sp->trace_id;
  pv.trace_end = sp->trace_end; pv.trace_tag = nullptr; pv.d = sp->d;
  pv.n_rows = (int32_t)sp->n_rows;

  // the counters and the query-valid flags must not carry over from the previous call
  e = cudaMemsetAsync(base + kStaticListBytes, 0, kStaticFlagBytes + sizeof(DeviceStats), st);
  if (e != cudaSuccess) {
    snprintf(g_static_err, sizeof g_static_err, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    return OILBIRD_ECUDA;
  }
  const int kk = list_len(pr->k);
  int32_t n_lists = 0;
  if (sp->n_rows > 0) {
    e = launch_scan_gemv(pv, (const uint16_t*)q_bf16, nq, pr->k, kk, nullptr, partial, q_valid,
                         stats, kStaticMaxLists, g_num_sms[sp->device], &n_lists, nullptr, st);
  } else {
    // nothing to scan: the flags only have to say whether each query is usable; the
    // merge kernel then reports "no neighbours" for all of them
    e = cudaMemsetAsync(q_valid, 0, sizeof(int32_t) * kStaticMaxNq, st);
  }
  if (e != cudaSuccess) {
    snprintf(g_static_err, sizeof g_static_err, "scan launch: %s", cudaGetErrorString(e));
    return OILBIRD_ECUDA;
  }
  e = launch_merge_gather(pv, partial, n_lists, nq, kk, q_valid, gp, *out, st);
  if (e != cudaSuccess) {
    snprintf(g_static_err, sizeof g_static_err, "merge launch: %s", cudaGetErrorString(e));
    return OILBIRD_ECUDA;
  }
  return OILBIRD_OK;
}

}  // extern "C"
