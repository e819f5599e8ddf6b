// The pool object behind the opaque handle of the C-ABI, shared by the files that implement
// entry points on it (pool.cu, index.cu).  Nothing here is visible outside the library.
#pragma once
#include <vector>

#include "internal.h"

namespace oilbird {

// Byte offsets of every device array inside one allocation.
constexpr int kMaxGuards = 24;
struct Layout {
  size_t keys, tok, trace_id, trace_end, trace_tag, trace_gbase, qn, q_valid, partial, stats;
  size_t xchg;
  size_t q_stage, ex_stage, st_stage, tok_stage, stage_end, fuse_ready, scales;
  size_t pipe_stage[2];      // two more staging blocks [q_stage, stage_end) for host steps in flight
  size_t total;
  // OILBIRD_DEBUG_GUARDS: sentinel bytes [g_lo, g_hi) behind every array (from its last
  // byte to the next array's first), named after the array they follow
  int n_guards;
  size_t g_lo[kMaxGuards], g_hi[kMaxGuards];
  const char* g_name[kMaxGuards];
};
constexpr unsigned char kGuardByte = 0xA5;

struct Resolved {
  int32_t d, max_traces, max_nq, max_k, max_append, max_lists;
  int32_t e4m3;              // keys are E4M3 codes with one scale per row
  int32_t guards;            // guard zones between the arrays (debugging aid)
  int64_t capacity;
};

}  // namespace oilbird

struct oilbird_pool {
  oilbird::Resolved r;
  oilbird::Layout lay;
  int device, num_sms;
  bool owns_mem;
  unsigned char* base;
  // device arrays
  uint16_t* keys;            // bf16 keys, or ...
  uint8_t* codes;            // ... E4M3 codes (the same memory) with ...
  float* scales;             // ... one scale per row
  int32_t *tok, *trace_id, *trace_end;
  uint64_t* trace_tag;
  int64_t* trace_gbase;      // global position of each trace's first row (row sharding)
  uint16_t* qn;
  int32_t* q_valid;
  unsigned long long* partial;
  oilbird::DeviceStats* stats;
  float* xchg;               // tensor scan: cross-CTA threshold exchange
  unsigned long long* fuse_ready;   // rows published by appends fused into a scan ...
  unsigned long long fuse_target;   // ... and the host's count of them (enqueue time)
  // host bookkeeping (enqueue-time truth)
  int64_t n_rows;
  std::vector<int64_t> t_start, t_end;
  std::vector<uint64_t> t_tag;
  std::vector<int64_t> t_gbase;     // global position of each trace's first row, or -1 if
                                    // it is simply the local one (pool is not a shard)
  int64_t launches;
  int64_t generation;         // counts the calls that renumber rows (reset, eviction)
  // profiling
  bool profile;
  std::vector<cudaEvent_t> ev;   // pairs
  int ev_used;
  // pinned staging for host variants
  unsigned char* pinned;       // host address
  unsigned char* pinned_dev;   // the same block as the device sees it
  size_t blob_off, result_off;   // of slot 0; slot s is slot_stride bytes further on
  size_t slot_stride;
  cudaEvent_t upload_done;
  bool upload_pending;
  // host steps: slots 0 and 1 belong to step_host_begin .. step_host_end (inputs uploaded
  // on copy_stream into a staging block of their own, so that the upload of one step runs
  // under the kernels of the step before it); the last slot serves the synchronous calls
  struct HostSlot { bool busy; int32_t nq, k, L; cudaEvent_t copied, done; } slot[3];
  cudaStream_t copy_stream;
  // tensor-core scan: TMA tensor maps of this pool (nullptr = path unavailable)
  size_t smem_limit;
  oilbird::TcCache* tc;
};

namespace oilbird {
// The kernels' view of a pool's arrays at its current size.
inline PoolView pool_view(const oilbird_pool* p) {
  PoolView pv;
  pv.keys = p->keys; pv.tok = p->tok; pv.trace_id = p->trace_id; pv.trace_end = p->trace_end;
  pv.trace_tag = p->trace_tag; pv.d = p->r.d; pv.n_rows = (int32_t)p->n_rows;
  return pv;
}
}  // namespace oilbird
