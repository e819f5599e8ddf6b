// Host-side interface between the C-ABI layer (pool.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/oilbird.h"

namespace oilbird {

__host__ __device__ inline int next_pow2(int v) {
  int p = 1;
  while (p < v) p <<= 1;
  return p;
}

// ---- programmatic launches ---------------------------------------------------------
// Whether this process may chain kernels with programmatic stream serialization at all:
// only when the driver loads modules eagerly (CUDA_MODULE_LOADING=EAGER before CUDA starts).
// With lazy loading, the first steps of a process were seen to dead-lock now and then on
// the largest configuration while kernels of the chain were resident and waiting; the
// mechanism inside the driver was never established, so under lazy loading (or when the
// mode cannot be read) every launch of the library is a plain one.  Evaluated once.
bool pdl_process_ok();
// Set by an entry point for the calls it is about to make: plain launches for this call
// (scans that run for milliseconds gain nothing from overlapping a 5 us neighbour).
extern thread_local bool tl_pdl_off;
struct PdlScope {
  bool prev;
  explicit PdlScope(bool off) : prev(tl_pdl_off) { tl_pdl_off = tl_pdl_off || off; }
  ~PdlScope() { tl_pdl_off = prev; }
};

// Launch, with programmatic stream serialization where the policy above allows it (see
// pdl_enter() in common.cuh; for a plain launch the kernel's griddepcontrol instructions
// are no-ops).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  const bool pdl = !tl_pdl_off && pdl_process_ok();
  cfg.attrs = pdl ? attr : nullptr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Everything a kernel needs before its first launch is done once per device, before any
// kernel of the library is launched there (oilbird_pool_create and the first use of the
// ring, merge, shard and static entry points): asking for a function's attributes loads
// it (with lazy module loading a kernel is otherwise loaded at its first launch, which can
// wait for the device to go idle), and kernels with dynamic shared memory get their limit
// raised to the device's maximum here instead of at every launch.
template <typename K>
inline cudaError_t preload_kernel(K kernel, bool dynamic_smem = false) {
  cudaFuncAttributes attr;
  cudaError_t e = cudaFuncGetAttributes(&attr, kernel);
  if (e != cudaSuccess || !dynamic_smem) return e;
  int dev = 0, optin = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
    return e;
  const int room = optin - (int)attr.sharedSizeBytes;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, room > 0 ? room : 0);
}
cudaError_t preload_append_kernels();
cudaError_t preload_evict_kernels();
cudaError_t preload_index_kernels();
cudaError_t preload_merge_kernels();
cudaError_t preload_merge_tree_kernels();
cudaError_t preload_quant8_kernels();
cudaError_t preload_ring_kernels();
cudaError_t preload_scan_gemv_kernels();
cudaError_t preload_scan_mma_kernels();
cudaError_t preload_scan_tc_kernels();
cudaError_t preload_shard_kernels();
// all of the above, once per device (the current device); thread-safe
cudaError_t preload_all_kernels();

// Device counters (one struct in device memory per pool).
struct DeviceStats {
  unsigned long long degenerate_rows;
  unsigned long long nonfinite_queries;
  int stalled;
  int pad;
  // how long a device-side wait may spin before it gives up, in nanoseconds of %globaltimer
  // (0 = kDefaultWaitNs); survives reset()
  unsigned long long wait_limit_ns;
};
constexpr unsigned long long kDefaultWaitNs = 2000000000ull;
constexpr size_t kStatsCounterBytes = 24;      // the part of DeviceStats that reset() clears

// Views of the pool's device arrays handed to the kernels.
struct PoolView {
  const uint16_t* keys;      // [capacity, d] bf16, row-major, normalised (Eq. 1)
  const int32_t* tok;        // [capacity]
  const int32_t* trace_id;   // [capacity]
  const int32_t* trace_end;  // [max_traces] one past the last row of each trace
  const uint64_t* trace_tag; // [max_traces]
  int32_t d;
  int32_t n_rows;            // rows visible to this launch
};

struct GatherParams {
  int32_t k, offset, depth_mode, cont_len, n_tiers;
  float theta;
  float tier_thr[OILBIRD_MAX_TIERS];
  int32_t tier_depth[OILBIRD_MAX_TIERS];
};

// Range checks of the retrieval parameters shared by every query entry point; fills gp.
int check_query_params(int32_t nq, int32_t max_nq, int32_t max_k, const oilbird_query_params* pr,
                       GatherParams* gp);

// The append of one serving step, done by the first n CTAs of the CUDA-core scan itself
// instead of by a kernel of its own (n == 0: nothing to append).  CTA i normalises row i
// into keys[row0 + i] and then adds one to *ready; a warp of the scan that is about to
// read a row >= row0 first waits (bounded) for *ready to reach `target`.
constexpr int kFuseMaxRows = 64;
struct FusedAppend {
  const uint16_t* states;       // [n, d] raw bf16
  const int32_t* tokens;        // [n]
  uint16_t* keys;
  int32_t* tok;
  int32_t* trace_id;
  int32_t* trace_end;
  uint64_t* trace_tag;
  int64_t* trace_gbase;
  unsigned long long* ready;    // rows published by fused appends since the pool was created
  unsigned long long target;    // value of *ready once this step's rows are all in
  uint64_t tag;
  int64_t gbase;
  int32_t n, row0, trace, set_tag;
};

// a1: normalise n raw bf16 rows into keys[row0..], store tokens / trace ids, and let one
// thread publish the trace-table entry (trace, end, tag).
cudaError_t launch_append(const uint16_t* states, const int32_t* tokens, int64_t n, int32_t d,
                          uint16_t* keys, int32_t* tok, int32_t* trace_id, int64_t row0,
                          int32_t trace, int32_t* trace_end, uint64_t* trace_tag, uint64_t tag,
                          int64_t* trace_gbase, int64_t gbase, int set_tag, DeviceStats* stats,
                          int32_t num_sms, cudaStream_t st);

// Row sharding over several pools: local rows -> caller-assigned global positions, and the
// merge of the shards' gathered query results (see shard.cu).
cudaError_t launch_to_global(const int32_t* idx, int64_t* out, int64_t n, const int32_t* trace_id,
                             const int32_t* trace_end, const int64_t* trace_gbase, int32_t n_rows,
                             cudaStream_t st);

// query preparation: qn[r] = bf16(q[r]/||q[r]||) for r < nq, zero rows up to nq_pad,
// q_valid[r] = 0 for a query holding NaN/Inf.
// Also fills xchg[0..n_xchg) with -inf (the tensor scan's threshold exchange, see scan_tc.cu)
// and zeroes the kTcXchgCounters words behind them.
// f16_scaled: qn holds f16(2^14 * bf16 value) instead (the tensor scan of 8-bit pools).
cudaError_t launch_qnorm(const uint16_t* q, int32_t nq, int32_t nq_pad, int32_t d, uint16_t* qn,
                         int32_t* q_valid, DeviceStats* stats, float* xchg, int32_t n_xchg,
                         bool f16_scaled, cudaStream_t st);

// Cross-CTA threshold exchange of the tensor scan: per query one published best score per
// CTA (kTcMaxCtas slots) followed by one agreed lower bound per query.
constexpr int kTcMaxCtas = 160;   // >= the 148 SMs of a B200; five values per lane
constexpr int kTcXchgFloats = OILBIRD_MAX_NQ * kTcMaxCtas + OILBIRD_MAX_NQ;
// ... followed by kTcXchgCounters words that the query preparation sets to zero: arrival
// counters of the two rendezvous in a CTA's first tile (see scan_tc.cu)
constexpr int kTcXchgCounters = 4;

// Length of the candidate lists exchanged between scan and merge for a given k.
inline int list_len(int k) { int p = next_pow2(k); return p < 32 ? 32 : p; }

// a2+a3 (CUDA cores): normalise the nq raw queries, score every row against them and
// leave, per CTA and query, a descending list of kk = list_len(k) packed candidates in
// partial[list][q][kk].  Also writes q_valid.  Returns the number of lists through *n_lists.
cudaError_t launch_scan_gemv(const PoolView& pv, const uint16_t* q_raw, int32_t nq, int32_t k,
                             int32_t kk, const uint64_t* exclude_tag, unsigned long long* partial,
                             int32_t* q_valid, DeviceStats* stats, int32_t max_lists,
                             int32_t num_sms, int32_t* n_lists, const FusedAppend* fused,
                             cudaStream_t st);

// The same two steps for pools with 8-bit keys (E4M3 codes, one fp32 scale per row).
cudaError_t launch_append_e4m3(const uint16_t* states, const int32_t* tokens, int64_t n, int32_t d,
                               uint8_t* codes, float* scales, int32_t* tok, int32_t* trace_id,
                               int64_t row0, int32_t trace, int32_t* trace_end,
                               uint64_t* trace_tag, uint64_t tag, int64_t* trace_gbase,
                               int64_t gbase, int set_tag, DeviceStats* stats, cudaStream_t st);
cudaError_t launch_scan_gemv_e4m3(const uint8_t* codes, const float* scales, const PoolView& pv,
                                  const uint16_t* q_raw, int32_t nq, int32_t k, int32_t kk,
                                  const uint64_t* exclude_tag, unsigned long long* partial,
                                  int32_t* q_valid, DeviceStats* stats, int32_t max_lists,
                                  int32_t num_sms, int32_t* n_lists, const FusedAppend* fused,
                                  cudaStream_t st);

// Eviction: move rows [head, head+live) of every per-row array down to [0, live) in place
// (cooperative launch; trace ids drop by n_traces).  scales may be nullptr.
cudaError_t launch_compact(unsigned char* keys, float* scales, int32_t* tok, int32_t* trace_id,
                           int64_t head, int64_t live, int64_t row_bytes, int32_t n_traces,
                           int32_t num_sms, cudaStream_t st);

// CTAs the CUDA-core scan launches for a pool of n_rows rows.
inline int32_t scan_gemv_grid(int64_t n_rows, int32_t num_sms, int32_t max_lists) {
  // at least 32 rows per CTA, at most two CTAs per SM
  int64_t want = (n_rows + 31) / 32;
  int32_t grid = (int32_t)(want < 1 ? 1 : (want > 2 * num_sms ? 2 * num_sms : want));
  return grid > max_lists ? max_lists : grid;
}

// a2+a3 (warp-level tensor cores, small batches): the same contract as the CUDA-core scan,
// eight or sixteen queries per pass over the keys.  Needs d % 128 == 0, kk <= 64 and room for the eight
// normalised queries in shared memory.
// (8-bit pools: codes and scales given, d % 256 == 0, f16 MMAs, no appended rows.)
bool scan_mma_supports(int32_t d, int32_t kk, size_t smem_limit, bool fp8);
// 8-query tiles per pass the kernel would use for nq queries (1 or 2; 0 = unsupported; with
// one tile and 16-bit keys it can append a step's rows itself), and the CTAs it launches
int scan_mma_tiles(int32_t d, int32_t kk, int32_t nq, size_t smem_limit, bool fp8);
int32_t scan_mma_grid(int64_t n_rows, int32_t num_sms, int32_t max_lists);
cudaError_t launch_scan_mma(const PoolView& pv, const uint8_t* codes, const float* scales,
                            const uint16_t* q_raw, int32_t nq, int32_t k, int32_t kk,
                            const uint64_t* exclude_tag, unsigned long long* partial,
                            int32_t* q_valid, DeviceStats* stats, int32_t max_lists,
                            int32_t num_sms, size_t smem_limit, int32_t* n_lists,
                            const FusedAppend* fused, cudaStream_t st);

// a2+a3 (tensor cores): the same contract for queries [q0, q0+nq_c) of a call whose
// normalised queries already sit in qn.  TcCache holds the pool's TMA tensor maps
// (nullptr from create = tensor path unavailable).
struct TcCache;
// fp8: `keys` are E4M3 codes (one byte per element); launch_scan_tc then wants the rows' scales
// and the queries in qn as f16 scaled by 2^14 (launch_qnorm's f16_scaled).
TcCache* tc_cache_create(const void* keys, int64_t capacity, int32_t d, const void* qn,
                         int64_t qn_rows, bool fp8);
void tc_cache_destroy(TcCache* cache);
int tc_queries_per_pass(int nq, int k, int n_rows, int num_sms, size_t smem_limit, bool fp8);
cudaError_t launch_scan_tc(TcCache* cache, const PoolView& pv, int32_t q0, int32_t nq_c,
                           int32_t nq_total, int32_t k, int32_t kk, const uint64_t* exclude_tag,
                           unsigned long long* partial, DeviceStats* stats, float* xchg,
                           int32_t num_sms, size_t smem_limit, int32_t* n_lists,
                           const float* scales, cudaStream_t st);

// Exercises the give-up path of the two kinds of device-side wait the library has (the
// fused append's row counter and an mbarrier of the tensor scan) on a counter nobody
// advances and a barrier nobody arrives at: both waits run out after the pool's wait limit,
// raise `stalled` and return.  One small CTA; nothing else is touched.
cudaError_t launch_stall_selftest(const unsigned long long* ready, DeviceStats* stats,
                                  cudaStream_t st);

// a3 (final merge) + a4 + a5 + a6: one CTA per query.
cudaError_t launch_merge_gather(const PoolView& pv, const unsigned long long* partial,
                                int32_t n_lists, int32_t nq, int32_t kk, const int32_t* q_valid,
                                const GatherParams& gp, const oilbird_query_out& out,
                                cudaStream_t st);

// a4 + a5 + a6 on caller-supplied neighbours.
cudaError_t launch_gather_only(const PoolView& pv, const int32_t* idx, const float* score,
                               int32_t nq, const GatherParams& gp, const oilbird_query_out& out,
                               cudaStream_t st);

}  // namespace oilbird
