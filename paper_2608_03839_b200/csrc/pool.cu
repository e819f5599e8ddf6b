// C-ABI layer: argument checks, memory layout of the pool in HBM, host-side trace
// bookkeeping and the launch sequence of each entry point.  No arithmetic of the
// method lives here.
#include <cuda.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <new>
#include <vector>

#include "internal.h"
#include "pool_priv.h"

using namespace oilbird;

static thread_local char g_cuda_err[256] = "";

namespace oilbird {
thread_local bool tl_pdl_off = false;

// The driver's module loading mode, read once (CUDA must be initialised: every caller has
// launched or is about to launch).  Anything but "eager" switches programmatic launches off.
bool pdl_process_ok() {
  static const bool ok = [] {
    typedef CUresult (*GetModeFn)(CUmoduleLoadingMode*);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuModuleGetLoadingMode", &fn, cudaEnableDefault, &qres) !=
            cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
      return false;
    CUmoduleLoadingMode mode;
    if (((GetModeFn)fn)(&mode) != CUDA_SUCCESS) return false;
    return mode == CU_MODULE_EAGER_LOADING;
  }();
  return ok;
}

cudaError_t preload_all_kernels() {
  static std::mutex mu;
  static bool done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
  if ((e = cudaFree(nullptr)) != cudaSuccess) return e;      // the context exists from here on
  (void)pdl_process_ok();
  if ((e = preload_append_kernels()) != cudaSuccess) return e;
  if ((e = preload_evict_kernels()) != cudaSuccess) return e;
  if ((e = preload_index_kernels()) != cudaSuccess) return e;
  if ((e = preload_merge_kernels()) != cudaSuccess) return e;
  if ((e = preload_merge_tree_kernels()) != cudaSuccess) return e;
  if ((e = preload_quant8_kernels()) != cudaSuccess) return e;
  if ((e = preload_ring_kernels()) != cudaSuccess) return e;
  if ((e = preload_scan_gemv_kernels()) != cudaSuccess) return e;
  if ((e = preload_scan_mma_kernels()) != cudaSuccess) return e;
  if ((e = preload_scan_tc_kernels()) != cudaSuccess) return e;
  if ((e = preload_shard_kernels()) != cudaSuccess) return e;
  if (dev >= 0 && dev < 64) done[dev] = true;
  return cudaSuccess;
}
}  // namespace oilbird


static int cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", what, cudaGetErrorString(e));
  return e == cudaErrorMemoryAllocation ? OILBIRD_ENOMEM : OILBIRD_ECUDA;
}
#define CU(call)                                          \
  do {                                                    \
    cudaError_t e_ = (call);                              \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call);   \
  } while (0)

namespace {
constexpr size_t kAlign = 256;
constexpr int kMaxProfile = 4096;
size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

bool resolve(const oilbird_pool_config* c, int num_sms, Resolved* r) {
  if (!c) return false;
  if (c->d < 8 || c->d > 16384 || (c->d % 8) != 0) return false;
  if (c->capacity_rows < 1 || c->capacity_rows > 2147483000LL) return false;
  if (c->flags & ~(uint32_t)(OILBIRD_KEYS_E4M3 | OILBIRD_DEBUG_GUARDS)) return false;
  r->e4m3 = (c->flags & OILBIRD_KEYS_E4M3) ? 1 : 0;
  r->guards = (c->flags & OILBIRD_DEBUG_GUARDS) ? 1 : 0;
  if (r->e4m3 && (c->d % 16) != 0) return false;      // 16 codes per 16-byte load
  r->d = c->d;
  r->capacity = c->capacity_rows;
  int64_t mt = c->max_traces > 0 ? c->max_traces
                                 : (c->capacity_rows < (1 << 20) ? c->capacity_rows : (1 << 20));
  if (c->max_traces < 0) return false;
  r->max_traces = (int32_t)mt;
  r->max_nq = c->max_nq > 0 ? c->max_nq : OILBIRD_MAX_NQ;
  r->max_k = c->max_k > 0 ? c->max_k : 64;
  r->max_append = c->max_append > 0 ? c->max_append : 4096;
  if (r->max_nq > OILBIRD_MAX_NQ || r->max_k > OILBIRD_MAX_K || c->max_nq < 0 || c->max_k < 0 ||
      c->max_append < 0)
    return false;
  r->max_lists = 2 * num_sms;
  return true;
}

Layout make_layout(const Resolved& r) {
  Layout L;
  size_t off = 0;
  L.n_guards = 0;
  bool guards = r.guards != 0;
  auto take = [&](size_t bytes, const char* name) {
    const size_t o = off;
    off = align_up(off + bytes);
    if (guards && L.n_guards < kMaxGuards) {
      L.g_lo[L.n_guards] = o + bytes;
      off += kAlign;                       // one more aligned block of sentinel bytes
      L.g_hi[L.n_guards] = off;
      L.g_name[L.n_guards++] = name;
    }
    return o;
  };
  const size_t nq_pad = (size_t)(r.max_nq + 15) / 16 * 16;
  const size_t k_pad = (size_t)list_len(r.max_k);
  L.keys = take((size_t)r.capacity * r.d * (r.e4m3 ? 1 : 2), "keys");
  L.scales = take(r.e4m3 ? (size_t)r.capacity * 4 : 0, "scales");
  L.tok = take((size_t)r.capacity * 4, "tokens");
  L.trace_id = take((size_t)r.capacity * 4, "trace ids");
  L.trace_end = take((size_t)r.max_traces * 4, "trace ends");
  L.trace_tag = take((size_t)r.max_traces * 8, "trace tags");
  L.trace_gbase = take((size_t)r.max_traces * 8, "trace global bases");
  L.qn = take(nq_pad * r.d * 2, "normalised queries");
  L.q_valid = take(nq_pad * 4, "query-valid flags");
  L.partial = take((size_t)r.max_lists * r.max_nq * k_pad * 8, "candidate lists");
  L.stats = take(sizeof(DeviceStats), "counters");
  L.fuse_ready = take(8, "fused-append counter");
  L.xchg = take((size_t)(kTcXchgFloats + kTcXchgCounters) * 4, "threshold exchange");
  // staging for the *_host variants (adjacent: query_host/step_host fill them with one copy)
  guards = false;                          // no sentinels inside the one-copy staging block
  L.q_stage = take((size_t)r.max_nq * r.d * 2, "");
  L.ex_stage = take((size_t)r.max_nq * 8, "");
  L.st_stage = take((size_t)r.max_append * r.d * 2, "");
  guards = r.guards != 0;
  L.tok_stage = take((size_t)r.max_append * 4, "host staging");
  L.stage_end = L.tok_stage + align_up((size_t)r.max_append * 4);   // (a guard may follow)
  const size_t stage_bytes = L.stage_end - L.q_stage;
  guards = false;
  L.pipe_stage[0] = take(stage_bytes, "");
  guards = r.guards != 0;
  L.pipe_stage[1] = take(stage_bytes, "staging of host steps in flight");
  L.total = off;
  return L;
}
}  // namespace

extern "C" {

const char* oilbird_strerror(int code) {
  switch (code) {
    case OILBIRD_OK: return "ok";
    case OILBIRD_EINVAL: return "invalid argument";
    case OILBIRD_ECAPACITY: return "pool capacity exceeded";
    case OILBIRD_ENOMEM: return "out of memory";
    case OILBIRD_ECUDA: return "CUDA error";
    case OILBIRD_ESTALL: return "a bounded device-side wait gave up";
    case OILBIRD_EGUARD: return "a guard zone of the pool's memory was overwritten";
    default: return "unknown error";
  }
}

const char* oilbird_last_cuda_error(void) { return g_cuda_err; }

void oilbird_query_params_default(oilbird_query_params* p) {
  if (!p) return;
  memset(p, 0, sizeof *p);
  p->k = 8;                 // Algorithm 1, Require line
  p->theta = 0.8f;          // Eq. 2
  p->offset = 2;            // Eq. 3: the chain starts at x_{i+2}
  p->depth_mode = OILBIRD_DEPTH_TIERED;
  p->cont_len = 48;
  p->n_tiers = 2;           // Eq. 3: D(s) = 48 if s >= 0.90; 8 if s >= 0.82; else 0
  p->tier_thr[0] = 0.90f; p->tier_depth[0] = 48;
  p->tier_thr[1] = 0.82f; p->tier_depth[1] = 8;
  p->exclude_tag = nullptr;
  p->path = OILBIRD_PATH_AUTO;
}

size_t oilbird_pool_arena_bytes(const oilbird_pool_config* cfg) {
  Resolved r;
  if (!resolve(cfg, 148, &r)) return 0;
  r.max_lists = 2 * 256;    // generous: the SM count is not known without the device
  return make_layout(r).total + kAlign;
}

int oilbird_pool_create(oilbird_pool_t** out, const oilbird_pool_config* cfg) {
  if (!out || !cfg) return OILBIRD_EINVAL;
  *out = nullptr;
  int n_dev = 0;
  CU(cudaGetDeviceCount(&n_dev));
  if (cfg->device < 0 || cfg->device >= n_dev) return OILBIRD_EINVAL;
  CU(cudaSetDevice(cfg->device));
  CU(preload_all_kernels());       // before anything of the library is launched on this device
  cudaDeviceProp prop;
  CU(cudaGetDeviceProperties(&prop, cfg->device));
  Resolved r;
  if (!resolve(cfg, prop.multiProcessorCount, &r)) return OILBIRD_EINVAL;
  Layout lay = make_layout(r);
  oilbird_pool* p = new (std::nothrow) oilbird_pool();
  if (!p) return OILBIRD_ENOMEM;
  p->r = r; p->lay = lay; p->device = cfg->device; p->num_sms = prop.multiProcessorCount;
  p->n_rows = 0; p->launches = 0; p->generation = 0; p->profile = false; p->ev_used = 0;
  p->pinned = nullptr; p->pinned_dev = nullptr;
  if (cfg->arena) {
    size_t mis = (size_t)((uintptr_t)cfg->arena % kAlign);
    size_t skip = mis ? kAlign - mis : 0;
    if (cfg->arena_bytes < lay.total + skip) { delete p; return OILBIRD_EINVAL; }
    p->base = (unsigned char*)cfg->arena + skip;
    p->owns_mem = false;
  } else {
    void* mem = nullptr;
    cudaError_t e = cudaMalloc(&mem, lay.total);
    if (e != cudaSuccess) { delete p; return cuda_fail(e, "cudaMalloc(pool)"); }
    p->base = (unsigned char*)mem;
    p->owns_mem = true;
  }
  p->keys = (uint16_t*)(p->base + lay.keys);
  p->codes = (uint8_t*)(p->base + lay.keys);
  p->scales = (float*)(p->base + lay.scales);
  p->tok = (int32_t*)(p->base + lay.tok);
  p->trace_id = (int32_t*)(p->base + lay.trace_id);
  p->trace_end = (int32_t*)(p->base + lay.trace_end);
  p->trace_tag = (uint64_t*)(p->base + lay.trace_tag);
  p->trace_gbase = (int64_t*)(p->base + lay.trace_gbase);
  p->qn = (uint16_t*)(p->base + lay.qn);
  p->q_valid = (int32_t*)(p->base + lay.q_valid);
  p->partial = (unsigned long long*)(p->base + lay.partial);
  p->stats = (DeviceStats*)(p->base + lay.stats);
  p->xchg = (float*)(p->base + lay.xchg);
  p->fuse_ready = (unsigned long long*)(p->base + lay.fuse_ready);
  p->fuse_target = 0;
  cudaError_t e = cudaMemset(p->stats, 0, sizeof(DeviceStats));
  if (e == cudaSuccess) e = cudaMemset(p->fuse_ready, 0, 8);
  for (int g = 0; g < lay.n_guards && e == cudaSuccess; ++g)
    e = cudaMemset(p->base + lay.g_lo[g], kGuardByte, lay.g_hi[g] - lay.g_lo[g]);
  if (e != cudaSuccess) {
    if (p->owns_mem) cudaFree(p->base);
    delete p;
    return cuda_fail(e, "cudaMemset(stats)");
  }
  p->smem_limit = prop.sharedMemPerBlockOptin;
  p->tc = (prop.major == 10) ? tc_cache_create(p->keys, r.capacity, r.d, p->qn,
                                             (r.max_nq + 15) / 16 * 16, r.e4m3 != 0)
                           : nullptr;
  *out = p;
  return OILBIRD_OK;
}

int oilbird_pool_destroy(oilbird_pool_t* p) {
  if (!p) return OILBIRD_EINVAL;
  cudaSetDevice(p->device);
  cudaDeviceSynchronize();
  for (cudaEvent_t e : p->ev) cudaEventDestroy(e);
  if (p->pinned) {
    cudaFreeHost(p->pinned);
    cudaEventDestroy(p->upload_done);
    for (auto& sl : p->slot) { cudaEventDestroy(sl.done); cudaEventDestroy(sl.copied); }
    cudaStreamDestroy(p->copy_stream);
  }
  tc_cache_destroy(p->tc);
  if (p->owns_mem) cudaFree(p->base);
  delete p;
  return OILBIRD_OK;
}

int oilbird_pool_reset(oilbird_pool_t* p, void* stream) {
  if (!p) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  CU(cudaMemsetAsync(p->stats, 0, kStatsCounterBytes, (cudaStream_t)stream));   // not the wait limit
  p->n_rows = 0;
  p->generation += 1;
  p->t_start.clear(); p->t_end.clear(); p->t_tag.clear(); p->t_gbase.clear();
  return OILBIRD_OK;
}

int64_t oilbird_pool_size(const oilbird_pool_t* p) { return p ? p->n_rows : 0; }
int32_t oilbird_pool_num_traces(const oilbird_pool_t* p) { return p ? (int32_t)p->t_start.size() : 0; }
int64_t oilbird_pool_launch_count(const oilbird_pool_t* p) { return p ? p->launches : 0; }

// The kernels read bf16 rows with 16-byte vector loads and the integer arrays word by word;
// a misaligned pointer would fault on the device, so it is turned away here.
static bool aligned(const void* p, uintptr_t a) { return ((uintptr_t)p & (a - 1)) == 0; }
static int misaligned(const char* what) {
  snprintf(g_cuda_err, sizeof g_cuda_err, "%s is not aligned as the header requires", what);
  return OILBIRD_EINVAL;
}

static int refused(const char* why) {
  snprintf(g_cuda_err, sizeof g_cuda_err, "%s", why);
  return OILBIRD_EINVAL;
}

// Scans of pools this large run for about a millisecond and more: chaining their kernels
// programmatically would gain a few microseconds on that, so they are launched plainly.
constexpr int64_t kPdlMaxKeyBytes = 4ll << 30;
static bool long_scan(const oilbird_pool* p) {
  return p->n_rows * (int64_t)p->r.d * (p->r.e4m3 ? 1 : 2) > kPdlMaxKeyBytes;
}

// Host side of an append: checks, then the trace bookkeeping (enqueue-time truth).
struct AppendPlan {
  bool open_new;
  int32_t trace;
  int64_t row0;
};

static int append_prepare(oilbird_pool_t* p, const void* states, const int32_t* tokens, int64_t n,
                          uint64_t tag, uint32_t flags, AppendPlan* ap, bool* nothing) {
  *nothing = false;
  if (!p || n < 0 || (n > 0 && (!states || !tokens))) return OILBIRD_EINVAL;
  if (n > 0 && !aligned(states, 16)) return misaligned("states");
  if (n > 0 && !aligned(tokens, 4)) return misaligned("tokens");
  ap->open_new = (flags & OILBIRD_NEW_TRACE) || p->t_start.empty();
  if (n == 0 && !ap->open_new) { *nothing = true; return OILBIRD_OK; }
  if (p->n_rows + n > p->r.capacity) return OILBIRD_ECAPACITY;
  if (ap->open_new && (int64_t)p->t_start.size() >= p->r.max_traces) return OILBIRD_ECAPACITY;
  if (ap->open_new) {
    p->t_start.push_back(p->n_rows);
    p->t_end.push_back(p->n_rows);
    p->t_tag.push_back(tag);
    p->t_gbase.push_back(-1);
  }
  ap->trace = (int32_t)p->t_start.size() - 1;
  ap->row0 = p->n_rows;
  return OILBIRD_OK;
}
static void append_rollback(oilbird_pool_t* p, const AppendPlan& ap) {
  if (ap.open_new) {
    p->t_start.pop_back(); p->t_end.pop_back(); p->t_tag.pop_back(); p->t_gbase.pop_back();
  }
  p->n_rows = ap.row0;
  if (!ap.open_new) p->t_end[ap.trace] = ap.row0;
}
static void append_commit(oilbird_pool_t* p, int64_t n, const AppendPlan& ap) {
  p->n_rows = ap.row0 + n;
  p->t_end[ap.trace] = p->n_rows;
}

// OILBIRD_EVICT_TO_FIT: how many of the oldest traces have to go so that n more rows (and a new
// trace, if one is opened) fit: the fewest, never the trace that is being extended.  Returns
// OILBIRD_ECAPACITY if even that does not make room.  *rows = the rows those traces hold.
static int evict_plan(const oilbird_pool* p, int64_t n, uint32_t flags, int32_t* n_traces,
                      int64_t* rows) {
  *n_traces = 0;
  *rows = 0;
  if (!(flags & OILBIRD_EVICT_TO_FIT)) return OILBIRD_OK;
  const bool open_new = (flags & OILBIRD_NEW_TRACE) || p->t_start.empty();
  const int32_t have = (int32_t)p->t_start.size();
  const int32_t may_go = open_new ? have : have - 1;          // the open trace stays
  int32_t nt = 0;
  int64_t dropped = 0;
  while ((p->n_rows - dropped + n > p->r.capacity ||
          (open_new && have - nt >= p->r.max_traces)) && nt < may_go) {
    dropped = p->t_end[nt];
    ++nt;
  }
  if (p->n_rows - dropped + n > p->r.capacity || (open_new && have - nt >= p->r.max_traces))
    return OILBIRD_ECAPACITY;
  *n_traces = nt;
  *rows = dropped;
  return OILBIRD_OK;
}
static int evict_to_fit(oilbird_pool_t* p, int64_t n, uint32_t flags, void* stream) {
  int32_t nt;
  int64_t rows;
  int rc = evict_plan(p, n, flags, &nt, &rows);
  if (rc || nt == 0) return rc;
  return oilbird_pool_evict_oldest(p, nt, nullptr, stream);
}

// global_row < 0: the pool is not a shard, a trace's global position is its local one.
static int append_impl(oilbird_pool_t* p, const void* states, const int32_t* tokens, int64_t n,
                       uint64_t tag, uint32_t flags, int64_t global_row, void* stream) {
  AppendPlan ap;
  bool nothing;
  if (!p || n < 0 || (n > 0 && (!states || !tokens))) return OILBIRD_EINVAL;
  int rc = evict_to_fit(p, n, flags, stream);
  if (rc) return rc;
  rc = append_prepare(p, states, tokens, n, tag, flags, &ap, &nothing);
  if (rc || nothing) return rc;
  CU(cudaSetDevice(p->device));
  PdlScope plain(long_scan(p));
  const int64_t gbase = global_row >= 0 ? global_row : ap.row0;
  cudaError_t e =
      p->r.e4m3
          ? launch_append_e4m3((const uint16_t*)states, tokens, n, p->r.d, p->codes, p->scales,
                               p->tok, p->trace_id, ap.row0, ap.trace, p->trace_end, p->trace_tag,
                               tag, p->trace_gbase, gbase, ap.open_new ? 1 : 0, p->stats,
                               (cudaStream_t)stream)
          : launch_append((const uint16_t*)states, tokens, n, p->r.d, p->keys, p->tok,
                          p->trace_id, ap.row0, ap.trace, p->trace_end, p->trace_tag, tag,
                          p->trace_gbase, gbase, ap.open_new ? 1 : 0, p->stats, p->num_sms,
                          (cudaStream_t)stream);
  if (e != cudaSuccess) {
    append_rollback(p, ap);
    return cuda_fail(e, "append kernel launch");
  }
  p->launches += 1;
  if (ap.open_new && global_row >= 0) p->t_gbase[ap.trace] = global_row;
  append_commit(p, n, ap);
  return OILBIRD_OK;
}

int oilbird_pool_evict_oldest(oilbird_pool_t* p, int32_t n_traces, int64_t* rows_dropped,
                              void* stream) {
  if (rows_dropped) *rows_dropped = 0;
  if (!p || n_traces < 0) return OILBIRD_EINVAL;
  const int32_t have = (int32_t)p->t_start.size();
  const int32_t nt = n_traces < have ? n_traces : have;
  if (nt == 0) return OILBIRD_OK;
  CU(cudaSetDevice(p->device));
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t head = p->t_end[nt - 1], live = p->n_rows - head;
  const int64_t row_bytes = p->r.e4m3 ? p->r.d : (int64_t)p->r.d * 2;
  cudaError_t e = launch_compact((unsigned char*)p->keys, p->r.e4m3 ? p->scales : nullptr, p->tok,
                                 p->trace_id, head, live, row_bytes, nt, p->num_sms, st);
  if (e != cudaSuccess) return cuda_fail(e, "compaction kernel launch");
  if (live > 0) p->launches += 1;
  p->generation += 1;
  // the host's copy of the trace table is the truth: renumber it, then publish it
  p->t_start.erase(p->t_start.begin(), p->t_start.begin() + nt);
  p->t_end.erase(p->t_end.begin(), p->t_end.begin() + nt);
  p->t_tag.erase(p->t_tag.begin(), p->t_tag.begin() + nt);
  p->t_gbase.erase(p->t_gbase.begin(), p->t_gbase.begin() + nt);
  const size_t left = p->t_start.size();
  std::vector<int32_t> ends(left);
  std::vector<int64_t> gb(left);
  for (size_t i = 0; i < left; ++i) {
    p->t_start[i] -= head;
    p->t_end[i] -= head;
    ends[i] = (int32_t)p->t_end[i];
    gb[i] = p->t_gbase[i] >= 0 ? p->t_gbase[i] : p->t_start[i];
  }
  p->n_rows = live;
  if (left > 0) {
    // pageable sources: each call returns once its source has been staged
    CU(cudaMemcpyAsync(p->trace_end, ends.data(), left * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(p->trace_tag, p->t_tag.data(), left * 8, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(p->trace_gbase, gb.data(), left * 8, cudaMemcpyHostToDevice, st));
  }
  if (rows_dropped) *rows_dropped = head;
  return OILBIRD_OK;
}

int oilbird_pool_append(oilbird_pool_t* p, const void* states, const int32_t* tokens, int64_t n,
                        uint64_t tag, uint32_t flags, void* stream) {
  return append_impl(p, states, tokens, n, tag, flags, -1, stream);
}

int oilbird_pool_append_global(oilbird_pool_t* p, const void* states, const int32_t* tokens,
                               int64_t n, uint64_t tag, uint32_t flags, int64_t global_row,
                               void* stream) {
  if (global_row < 0) return OILBIRD_EINVAL;
  return append_impl(p, states, tokens, n, tag, flags, global_row, stream);
}

int oilbird_pool_to_global(oilbird_pool_t* p, const int32_t* idx, int64_t* global_idx, int64_t n,
                           void* stream) {
  if (!p || n < 0 || (n > 0 && (!idx || !global_idx))) return OILBIRD_EINVAL;
  if (n == 0) return OILBIRD_OK;
  CU(cudaSetDevice(p->device));
  cudaError_t e = launch_to_global(idx, global_idx, n, p->trace_id, p->trace_end, p->trace_gbase,
                                   (int32_t)p->n_rows, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "to_global kernel launch");
  p->launches += 1;
  return OILBIRD_OK;
}

}  // extern "C"

namespace oilbird {
int check_query_params(int32_t nq, int32_t max_nq, int32_t max_k, const oilbird_query_params* pr,
                       GatherParams* gp) {
  if (!pr) return OILBIRD_EINVAL;
  if (nq < 1 || nq > max_nq) return OILBIRD_EINVAL;
  if (pr->k < 1 || pr->k > max_k) return OILBIRD_EINVAL;
  if (pr->cont_len < 1 || pr->cont_len > OILBIRD_MAX_CONT_LEN) return OILBIRD_EINVAL;
  if (pr->offset < 0 || pr->offset > (1 << 20)) return OILBIRD_EINVAL;
  if (pr->depth_mode != OILBIRD_DEPTH_FIXED && pr->depth_mode != OILBIRD_DEPTH_TIERED &&
      pr->depth_mode != OILBIRD_DEPTH_RANKED)
    return OILBIRD_EINVAL;
  if (pr->n_tiers < 0 || pr->n_tiers > OILBIRD_MAX_TIERS) return OILBIRD_EINVAL;
  if (pr->path < OILBIRD_PATH_AUTO || pr->path > OILBIRD_PATH_MMA) return OILBIRD_EINVAL;
  if (isnan(pr->theta)) return OILBIRD_EINVAL;
  gp->k = pr->k; gp->offset = pr->offset; gp->depth_mode = pr->depth_mode;
  gp->cont_len = pr->cont_len; gp->n_tiers = pr->n_tiers; gp->theta = pr->theta;
  for (int t = 0; t < OILBIRD_MAX_TIERS; ++t) {
    gp->tier_thr[t] = t < pr->n_tiers ? pr->tier_thr[t] : INFINITY;
    gp->tier_depth[t] = t < pr->n_tiers ? pr->tier_depth[t] : 0;
    if (t < pr->n_tiers && (isnan(pr->tier_thr[t]) || pr->tier_depth[t] < 0)) return OILBIRD_EINVAL;
  }
  return OILBIRD_OK;
}
}  // namespace oilbird

extern "C" {

static int check_params(const oilbird_pool* p, int32_t nq, const oilbird_query_params* pr,
                        GatherParams* gp) {
  return check_query_params(nq, p->r.max_nq, p->r.max_k, pr, gp);
}

static PoolView view_of(const oilbird_pool* p) { return pool_view(p); }

static bool out_ok(const oilbird_query_out* o, bool need_idx) {
  if (!o || !o->fired || !o->cont_len || !o->cont_tok) return false;
  if (!aligned(o->fired, 4) || !aligned(o->cont_len, 4) || !aligned(o->cont_tok, 4)) return false;
  if (!need_idx) return true;
  return o->idx && o->score && aligned(o->idx, 4) && aligned(o->score, 4);
}

// Key bytes up to which a batch of 3 to 16 queries goes to the warp-level tensor scan: it
// streams keys like the CUDA-core scan and starts within a few microseconds; above, the
// tcgen05 scan's higher streaming rate has made up for its ~40 us of start-up.
constexpr int64_t kMmaMaxKeyBytes = 2ll << 30;
// 9 to 16 queries (two 8-query tiles per pass, one CTA per SM) stream at two thirds of that
// rate: only pools that the start-up dominates (8,192 rows x 4096: 33 us against 53)
constexpr int64_t kMma16MaxKeyBytes = 128ll << 20;

// 8-bit pools: more than 8 queries go to the tcgen05 scan from this many bytes of codes on
constexpr int64_t kFp8TensorMinBytes = 32ll << 20;

static int resolve_path(const oilbird_pool* p, const oilbird_query_params* pr, int32_t nq,
                        int64_t n_rows) {
  // single-request decode streams keys through the CUDA cores; batches go to tcgen05,
  // small batches on pools of the paper's size to mma.sync
  if (pr->path != OILBIRD_PATH_AUTO) return pr->path;
  // (two queries on an 8-bit pool: the CUDA-core scan converts every code once per query and
  // is bound by that, 78 us against 63 at 268 MB of codes; below 128 MB its fused append
  // makes up for it)
  // (two queries on a 16-bit pool of 4 GB and more: the tcgen05 scan streams 4-5 % faster than
  // two FMAs per key element on the CUDA cores; C4 1.305 ms against 1.365, C5 2.54 against 2.63)
  if (nq == 2 && !p->r.e4m3 && p->tc && n_rows * (int64_t)p->r.d * 2 >= (4ll << 30))
    return OILBIRD_PATH_TENSOR;
  if (nq <= 1 || (nq == 2 && !(p->r.e4m3 && n_rows * (int64_t)p->r.d >= (128ll << 20))))
    return OILBIRD_PATH_GEMV;
  if (p->r.e4m3) {
    // 8-bit pools: the warp-level tensor scan scores 8 queries per pass over the codes (the
    // CUDA-core scan two); larger batches take the tcgen05 scan, which turns the codes into
    // f16 on the way and reads them once for the whole batch
    if (nq > 8 && p->tc && n_rows * (int64_t)p->r.d >= kFp8TensorMinBytes) return OILBIRD_PATH_TENSOR;
    return scan_mma_tiles(p->r.d, list_len(pr->k), nq, p->smem_limit, true) ? OILBIRD_PATH_MMA
                                                                             : OILBIRD_PATH_GEMV;
  }
  const int64_t key_bytes = n_rows * (int64_t)p->r.d * 2;
  const int64_t mma_max = nq > 8 ? kMma16MaxKeyBytes : kMmaMaxKeyBytes;
  if (nq <= 16 && key_bytes <= mma_max) {
    // up to 8 queries in one pass of 8; 9 to 16 only where 16 fit in one pass
    const int nt = scan_mma_tiles(p->r.d, list_len(pr->k), nq, p->smem_limit, false);
    if (nt == 2 || (nt == 1 && nq <= 8)) return OILBIRD_PATH_MMA;
  }
  return OILBIRD_PATH_TENSOR;
}

// Everything about a query that can be refused, checked before anything is enqueued (and,
// for a step, before anything is appended): arguments, parameters, and whether the scan the
// call resolves to exists for this pool.  Returns the scan through *path.
static int check_query(const oilbird_pool* p, const void* q, int32_t nq,
                       const oilbird_query_params* pr, const oilbird_query_out* out,
                       int64_t n_rows, GatherParams* gp, int* path) {
  if (!p || !q || !out_ok(out, true)) return OILBIRD_EINVAL;
  if (!aligned(q, 16)) return misaligned("q");
  int rc = check_params(p, nq, pr, gp);
  if (rc) return rc;
  if (pr->exclude_tag && !aligned(pr->exclude_tag, 8)) return misaligned("exclude_tag");
  *path = resolve_path(p, pr, nq, n_rows);     // n_rows: the pool's size when the scan runs
  if (*path == OILBIRD_PATH_MMA &&
      !scan_mma_supports(p->r.d, list_len(pr->k), p->smem_limit, p->r.e4m3))
    return OILBIRD_EINVAL;
  if (*path == OILBIRD_PATH_TENSOR && !p->tc) {
    snprintf(g_cuda_err, sizeof g_cuda_err, "tensor-core scan unavailable on this device");
    return OILBIRD_ECUDA;
  }
  return OILBIRD_OK;
}

// fused: the step's append, to be done by the CUDA-core scan itself (the rows are already
// counted in p->n_rows), or nullptr.
static int query_impl(oilbird_pool_t* p, const void* q, int32_t nq, const oilbird_query_params* pr,
                      const oilbird_query_out* out, void* stream, const FusedAppend* fused) {
  GatherParams gp;
  int path = 0;
  int rc = check_query(p, q, nq, pr, out, p ? p->n_rows : 0, &gp, &path);
  if (rc) return rc;
  CU(cudaSetDevice(p->device));
  PdlScope plain(long_scan(p));
  cudaStream_t st = (cudaStream_t)stream;
  const int kk = list_len(pr->k);
  const int nq_pad = (nq + 15) / 16 * 16;
  PoolView pv = view_of(p);
  cudaError_t e;

  int32_t n_lists = 0;
  if (p->n_rows == 0) {
    // nothing to scan: only classify the queries (a NaN/Inf query is still counted)
    e = launch_qnorm((const uint16_t*)q, nq, nq_pad, p->r.d, p->qn, p->q_valid, p->stats,
                     nullptr, 0, false, st);
    if (e != cudaSuccess) return cuda_fail(e, "qnorm kernel launch");
    p->launches += 1;
  } else {
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (p->profile && p->ev_used + 2 <= (int)p->ev.size()) {
      e0 = p->ev[p->ev_used]; e1 = p->ev[p->ev_used + 1];
      CU(cudaEventRecord(e0, st));
    }
    if (path == OILBIRD_PATH_TENSOR) {
      // (8-bit pools: the queries as f16 scaled by 2^14, the rows' scales applied to the scores)
      e = launch_qnorm((const uint16_t*)q, nq, nq_pad, p->r.d, p->qn, p->q_valid, p->stats,
                       p->xchg, kTcXchgFloats, p->r.e4m3 != 0, st);
      if (e != cudaSuccess) return cuda_fail(e, "qnorm kernel launch");
      p->launches += 1;
      // as many queries per pass as shared memory allows next to a 3-stage ring
      const int per_pass = tc_queries_per_pass(nq, pr->k, pv.n_rows, p->num_sms, p->smem_limit,
                                               p->r.e4m3 != 0);
      for (int q0 = 0; q0 < nq; q0 += per_pass) {
        const int nq_c = nq - q0 < per_pass ? nq - q0 : per_pass;
        e = launch_scan_tc(p->tc, pv, q0, nq_c, nq, pr->k, kk, pr->exclude_tag, p->partial,
                           p->stats, p->xchg, p->num_sms, p->smem_limit, &n_lists,
                           p->r.e4m3 ? p->scales : nullptr, st);
        if (e != cudaSuccess) return cuda_fail(e, "tensor scan kernel launch");
        p->launches += 1;
      }
    } else if (p->r.e4m3 && path == OILBIRD_PATH_MMA) {
      e = launch_scan_mma(pv, p->codes, p->scales, (const uint16_t*)q, nq, pr->k, kk,
                          pr->exclude_tag, p->partial, p->q_valid, p->stats, p->r.max_lists,
                          p->num_sms, p->smem_limit, &n_lists, fused, st);
      if (e != cudaSuccess) return cuda_fail(e, "8-bit warp-level tensor scan kernel launch");
      p->launches += 1;
    } else if (p->r.e4m3) {
      e = launch_scan_gemv_e4m3(p->codes, p->scales, pv, (const uint16_t*)q, nq, pr->k, kk,
                                pr->exclude_tag, p->partial, p->q_valid, p->stats, p->r.max_lists,
                                p->num_sms, &n_lists, fused, st);
      if (e != cudaSuccess) return cuda_fail(e, "8-bit scan kernel launch");
      p->launches += 1;
    } else if (path == OILBIRD_PATH_GEMV) {
      e = launch_scan_gemv(pv, (const uint16_t*)q, nq, pr->k, kk, pr->exclude_tag, p->partial,
                           p->q_valid, p->stats, p->r.max_lists, p->num_sms, &n_lists, fused, st);
      if (e != cudaSuccess) return cuda_fail(e, "scan kernel launch");
      p->launches += 1;
    } else if (path == OILBIRD_PATH_MMA) {
      e = launch_scan_mma(pv, nullptr, nullptr, (const uint16_t*)q, nq, pr->k, kk, pr->exclude_tag, p->partial,
                          p->q_valid, p->stats, p->r.max_lists, p->num_sms, p->smem_limit,
                          &n_lists, fused, st);
      if (e != cudaSuccess) return cuda_fail(e, "warp-level tensor scan kernel launch");
      p->launches += 1;
    } else {
      return OILBIRD_EINVAL;                   // (resolve_path names one of the scans above)
    }
    if (e0) {
      CU(cudaEventRecord(e1, st));
      p->ev_used += 2;
    }
  }
  e = launch_merge_gather(pv, p->partial, n_lists, nq, kk, p->q_valid, gp, *out, st);
  if (e != cudaSuccess) return cuda_fail(e, "merge kernel launch");
  p->launches += 1;
  return OILBIRD_OK;
}

int oilbird_pool_query(oilbird_pool_t* p, const void* q, int32_t nq,
                       const oilbird_query_params* pr, const oilbird_query_out* out,
                       void* stream) {
  return query_impl(p, q, nq, pr, out, stream, nullptr);
}

// Append + query.  For the single-request path and a handful of rows the append is done by
// the scan kernel itself (no kernel of its own in front of the scan).
static int step_impl(oilbird_pool_t* p, const void* states, const int32_t* tokens, int64_t n,
                     uint64_t tag, uint32_t flags, const void* q, int32_t nq,
                     const oilbird_query_params* pr, const oilbird_query_out* out, void* stream) {
  GatherParams gp;
  int path = 0;
  // nothing is appended if the query would be refused (arguments, parameters, or a scan this
  // pool does not have)
  if (!p) return OILBIRD_EINVAL;
  // (a step that evicts to make room: planned first, done only once the query has passed)
  int32_t evict_traces = 0;
  int64_t evict_rows = 0;
  int rc = evict_plan(p, n, flags, &evict_traces, &evict_rows);
  if (rc) return rc;
  const int64_t rows_after = p->n_rows - evict_rows + n;
  rc = check_query(p, q, nq, pr, out, rows_after, &gp, &path);
  if (rc) return rc;
  if (evict_traces > 0) {
    rc = oilbird_pool_evict_oldest(p, evict_traces, nullptr, stream);
    if (rc) return rc;
  }
  // (8-bit pools always use the CUDA-core scan; its passes beyond the first two queries
  // would find the rows in place, but keep to the single-request case there too)
  const bool gemv = p->r.e4m3 ? (nq <= 2 && path == OILBIRD_PATH_GEMV) : path == OILBIRD_PATH_GEMV;
  // the warp-level tensor scan appends the step's rows itself in its 8-query form (eight rows
  // per CTA on 16-bit keys, one on 8-bit keys)
  const bool mma8 = path == OILBIRD_PATH_MMA &&
                    scan_mma_tiles(p->r.d, list_len(pr->k), nq, p->smem_limit, p->r.e4m3) == 1;
  const bool fuse =
      n >= 1 && n <= kFuseMaxRows &&
      ((gemv && scan_gemv_grid(rows_after, p->num_sms, p->r.max_lists) >= n) ||
       (mma8 && (p->r.e4m3 ? 1 : 8) * (int64_t)scan_mma_grid(rows_after, p->num_sms, p->r.max_lists) >= n));
  if (!fuse) {
    rc = append_impl(p, states, tokens, n, tag, flags, -1, stream);
    if (rc) return rc;
    return query_impl(p, q, nq, pr, out, stream, nullptr);
  }
  AppendPlan ap;
  bool nothing;
  rc = append_prepare(p, states, tokens, n, tag, flags, &ap, &nothing);
  if (rc) return rc;
  FusedAppend fa;
  fa.states = (const uint16_t*)states; fa.tokens = tokens;
  fa.keys = p->keys; fa.tok = p->tok; fa.trace_id = p->trace_id; fa.trace_end = p->trace_end;
  fa.trace_tag = p->trace_tag; fa.trace_gbase = p->trace_gbase;
  fa.ready = p->fuse_ready; fa.target = p->fuse_target + (unsigned long long)n;
  fa.tag = tag; fa.gbase = ap.row0;
  fa.n = (int32_t)n; fa.row0 = (int32_t)ap.row0; fa.trace = ap.trace; fa.set_tag = ap.open_new ? 1 : 0;
  append_commit(p, n, ap);                        // the scan must see the new rows
  const int64_t launches_before = p->launches;
  rc = query_impl(p, q, nq, pr, out, stream, &fa);
  if (p->launches == launches_before) {           // the scan was never launched: no append either
    append_rollback(p, ap);
    return rc;
  }
  p->fuse_target = fa.target;
  return rc;
}

int oilbird_pool_step(oilbird_pool_t* p, const void* states, const int32_t* tokens, int64_t n,
                      uint64_t tag, uint32_t flags, const void* q, int32_t nq,
                      const oilbird_query_params* pr, const oilbird_query_out* out, void* stream) {
  if (n < 0 || (n > 0 && (!states || !tokens))) return OILBIRD_EINVAL;
  return step_impl(p, states, tokens, n, tag, flags, q, nq, pr, out, stream);
}

int oilbird_pool_gather(oilbird_pool_t* p, const int32_t* idx, const float* score, int32_t nq,
                        const oilbird_query_params* pr, const oilbird_query_out* out,
                        void* stream) {
  if (!p || !idx || !score || !out_ok(out, false)) return OILBIRD_EINVAL;
  if (!aligned(idx, 4) || !aligned(score, 4)) return misaligned("idx / score");
  GatherParams gp;
  int rc = check_params(p, nq, pr, &gp);
  if (rc) return rc;
  CU(cudaSetDevice(p->device));
  cudaError_t e = launch_gather_only(view_of(p), idx, score, nq, gp, *out, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "gather kernel launch");
  p->launches += 1;
  return OILBIRD_OK;
}

// ---- host-buffer variants ---------------------------------------------------------

// Pinned, device-mapped host staging: [append_host block | upload blob | result block].
// The append_host block is reused by the next append_host call, so an event marks when its
// upload has finished.  query_host and step_host return only after everything has
// completed; they pack their inputs into the upload blob (one host->device copy per call)
// and let the merge kernel write the results straight into the mapped result block, which
// is valid on the host once the stream has been synchronised.
constexpr size_t kPackLimit = 256 << 10;   // bytes up to which a step's inputs are packed
constexpr int kHostSlots = OILBIRD_HOST_SLOTS;   // host steps that may be in flight

struct HostBlob {
  size_t o_st, o_tok, o_q, o_ex, used;
};
static HostBlob blob_layout(const oilbird_pool* p, int64_t n, int32_t nq, bool with_ex) {
  HostBlob b;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  b.o_st = take((size_t)n * p->r.d * 2);
  b.o_tok = take((size_t)n * 4);
  b.o_q = take((size_t)nq * p->r.d * 2);
  b.o_ex = take(with_ex ? (size_t)nq * 8 : 0);
  b.used = off;
  return b;
}

static int ensure_pinned(oilbird_pool* p) {
  if (p->pinned) return OILBIRD_OK;
  const size_t a_bytes = (size_t)p->r.max_append * p->r.d * 2 + (size_t)p->r.max_append * 4;
  const size_t b_bytes = blob_layout(p, p->r.max_append, p->r.max_nq, true).used;
  const size_t o_bytes =
      (size_t)p->r.max_nq * ((size_t)p->r.max_k * (8 + 4 + 4 * OILBIRD_MAX_CONT_LEN) + 4);
  unsigned char* h = nullptr;
  // page-locking memory is a device-wide operation of the driver: let the device go idle
  // first rather than have it happen under kernels that are chained and waiting
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
  const size_t stride = align_up(b_bytes + o_bytes);
  e = cudaHostAlloc((void**)&h, align_up(a_bytes) + (kHostSlots + 1) * stride, cudaHostAllocMapped);
  if (e != cudaSuccess) return cuda_fail(e, "cudaHostAlloc");
  void* dptr = nullptr;
  e = cudaHostGetDevicePointer(&dptr, h, 0);
  // events and the copy stream; whatever was created is destroyed again if one of them fails
  cudaEvent_t made[1 + 2 * (kHostSlots + 1)];
  int n_made = 0;
  auto make_event = [&](cudaEvent_t* ev) {
    if (e != cudaSuccess) return;
    e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
    if (e == cudaSuccess) made[n_made++] = *ev;
  };
  make_event(&p->upload_done);
  for (auto& sl : p->slot) {
    sl.busy = false;
    make_event(&sl.done);
    make_event(&sl.copied);
  }
  // (non-blocking: no implicit ordering against the legacy default stream a caller may use)
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking);
  if (e != cudaSuccess) {
    for (int i = 0; i < n_made; ++i) cudaEventDestroy(made[i]);
    cudaFreeHost(h);
    return cuda_fail(e, "pinned staging set-up");
  }
  p->pinned = h;
  p->pinned_dev = (unsigned char*)dptr;
  p->blob_off = align_up(a_bytes);
  p->result_off = p->blob_off + b_bytes;
  p->slot_stride = stride;
  p->upload_pending = false;
  return OILBIRD_OK;
}

int oilbird_pool_append_host(oilbird_pool_t* p, const void* states, const int32_t* tokens,
                             int64_t n, uint64_t tag, uint32_t flags, void* stream) {
  if (!p || n < 0 || n > p->r.max_append || (n > 0 && (!states || !tokens))) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  int rc = ensure_pinned(p);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  uint16_t* d_st = (uint16_t*)(p->base + p->lay.st_stage);
  int32_t* d_tok = (int32_t*)(p->base + p->lay.tok_stage);
  if (n > 0) {
    // The caller's buffers are free again when this returns: they are copied into pinned
    // staging first.  Device-side staging is reused in stream order.
    if (p->upload_pending) { CU(cudaEventSynchronize(p->upload_done)); p->upload_pending = false; }
    const size_t sb = (size_t)n * p->r.d * 2, tb = (size_t)n * 4;
    unsigned char* h_tok = p->pinned + (size_t)p->r.max_append * p->r.d * 2;
    memcpy(p->pinned, states, sb);
    memcpy(h_tok, tokens, tb);
    CU(cudaMemcpyAsync(d_st, p->pinned, sb, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(d_tok, h_tok, tb, cudaMemcpyHostToDevice, st));
    CU(cudaEventRecord(p->upload_done, st));
    p->upload_pending = true;
  }
  return oilbird_pool_append(p, d_st, d_tok, n, tag, flags, stream);
}

// Result block of a slot: idx | score | cont_len | cont_tok | fired.
struct HostResult {
  size_t o_idx, o_score, o_len, o_tok, o_fired;
};
static HostResult result_layout(size_t nq, size_t k, size_t L) {
  HostResult r;
  r.o_idx = 0;
  r.o_score = r.o_idx + nq * k * 4;
  r.o_len = r.o_score + nq * k * 4;
  r.o_tok = r.o_len + nq * k * 4;
  r.o_fired = r.o_tok + nq * k * L * 4;
  return r;
}

// First half of a host step (query_host: n = 0 and no append): inputs into the slot's
// pinned blob, one upload, the kernels, the results written by the merge kernel straight
// into the slot's mapped result block, an event behind them.  `direct` (the synchronous
// calls only) lets a large step upload from the caller's buffers instead of packing.
static int host_begin(oilbird_pool_t* p, bool do_append, const void* states, const int32_t* tokens,
                      int64_t n, uint64_t tag, uint32_t flags, const void* q, int32_t nq,
                      const oilbird_query_params* pr, int slot, void* stream) {
  if (!p || !q || slot < 0 || slot > kHostSlots) return OILBIRD_EINVAL;
  const bool direct = slot == kHostSlots;      // the synchronous calls' own slot
  if (n < 0 || n > p->r.max_append || (n > 0 && (!states || !tokens))) return OILBIRD_EINVAL;
  GatherParams gp;
  int rc = check_params(p, nq, pr, &gp);
  if (rc) return rc;
  CU(cudaSetDevice(p->device));
  rc = ensure_pinned(p);
  if (rc) return rc;
  if (p->slot[slot].busy) return refused("host slot still in flight (step_host_end not called)");
  cudaStream_t st = (cudaStream_t)stream;
  const size_t k = pr->k, L = pr->cont_len;

  // inputs: one packed block, one copy (the device staging areas are adjacent in the arena
  // and are reused in stream order, which is why all host calls of a pool share a stream)
  const HostBlob b = blob_layout(p, n, nq, pr->exclude_tag != nullptr);
  unsigned char* h_blob = p->pinned + p->blob_off + (size_t)slot * p->slot_stride;
  unsigned char* d_blob = p->base + (direct ? p->lay.q_stage : p->lay.pipe_stage[slot]);
  if (b.used > p->lay.stage_end - p->lay.q_stage) return OILBIRD_EINVAL;   // cannot happen
  oilbird_query_params dp = *pr;
  if (pr->exclude_tag) dp.exclude_tag = (const uint64_t*)(d_blob + b.o_ex);
  if (b.used <= kPackLimit || !direct) {
    // pack, one copy (for a small step a copy's fixed cost outweighs the host-side memcpy;
    // a step that stays in flight must not depend on the caller's buffers)
    if (n > 0) {
      memcpy(h_blob + b.o_st, states, (size_t)n * p->r.d * 2);
      memcpy(h_blob + b.o_tok, tokens, (size_t)n * 4);
    }
    memcpy(h_blob + b.o_q, q, (size_t)nq * p->r.d * 2);
    if (pr->exclude_tag) memcpy(h_blob + b.o_ex, pr->exclude_tag, (size_t)nq * 8);
    if (direct) {
      CU(cudaMemcpyAsync(d_blob, h_blob, b.used, cudaMemcpyHostToDevice, st));
    } else {
      // the slot's own staging block was last read by the step `end` has already waited
      // for, so the upload need not queue behind the kernels of the step before this one
      CU(cudaMemcpyAsync(d_blob, h_blob, b.used, cudaMemcpyHostToDevice, p->copy_stream));
      CU(cudaEventRecord(p->slot[slot].copied, p->copy_stream));
      CU(cudaStreamWaitEvent(st, p->slot[slot].copied, 0));
    }
  } else {
    // large synchronous step: the call synchronises before it returns, so the caller's
    // buffers are uploaded directly (DMA from pinned memory; the driver stages pageable
    // memory itself)
    cudaError_t ce = cudaSuccess;
    if (n > 0) {
      ce = cudaMemcpyAsync(d_blob + b.o_st, states, (size_t)n * p->r.d * 2, cudaMemcpyHostToDevice, st);
      if (ce == cudaSuccess)
        ce = cudaMemcpyAsync(d_blob + b.o_tok, tokens, (size_t)n * 4, cudaMemcpyHostToDevice, st);
    }
    if (ce == cudaSuccess)
      ce = cudaMemcpyAsync(d_blob + b.o_q, q, (size_t)nq * p->r.d * 2, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess && pr->exclude_tag)
      ce = cudaMemcpyAsync(d_blob + b.o_ex, pr->exclude_tag, (size_t)nq * 8, cudaMemcpyHostToDevice, st);
    if (ce != cudaSuccess) {
      cudaStreamSynchronize(st);             // nothing may still read the caller's buffers
      return cuda_fail(ce, "cudaMemcpyAsync(host step)");
    }
  }

  const HostResult o = result_layout(nq, k, L);
  unsigned char* d_out = p->pinned_dev + p->result_off + (size_t)slot * p->slot_stride;
  oilbird_query_out dout;
  dout.idx = (int32_t*)(d_out + o.o_idx);
  dout.score = (float*)(d_out + o.o_score);
  dout.cont_len = (int32_t*)(d_out + o.o_len);
  dout.cont_tok = (int32_t*)(d_out + o.o_tok);
  dout.fired = (int32_t*)(d_out + o.o_fired);
  if (do_append)
    rc = step_impl(p, d_blob + b.o_st, (const int32_t*)(d_blob + b.o_tok), n, tag, flags,
                   d_blob + b.o_q, nq, &dp, &dout, stream);
  else
    rc = query_impl(p, d_blob + b.o_q, nq, &dp, &dout, stream, nullptr);
  if (rc) {
    cudaStreamSynchronize(st);               // also frees the caller's buffers on error
    return rc;
  }
  CU(cudaEventRecord(p->slot[slot].done, st));
  p->slot[slot].busy = true;
  p->slot[slot].nq = nq; p->slot[slot].k = (int32_t)k; p->slot[slot].L = (int32_t)L;
  return OILBIRD_OK;
}

// Second half: wait for the slot's event, hand the results over.
static int host_end(oilbird_pool_t* p, int slot, const oilbird_query_out* out) {
  if (!p || slot < 0 || slot > kHostSlots || !out_ok(out, true)) return OILBIRD_EINVAL;
  if (!p->pinned || !p->slot[slot].busy) return refused("no host step in flight in this slot");
  CU(cudaSetDevice(p->device));
  p->slot[slot].busy = false;
  cudaError_t e = cudaEventSynchronize(p->slot[slot].done);
  if (e != cudaSuccess) return cuda_fail(e, "cudaEventSynchronize");
  const size_t nq = p->slot[slot].nq, k = p->slot[slot].k, L = p->slot[slot].L;
  const HostResult o = result_layout(nq, k, L);
  const unsigned char* h_out = p->pinned + p->result_off + (size_t)slot * p->slot_stride;
  memcpy(out->idx, h_out + o.o_idx, nq * k * 4);
  memcpy(out->score, h_out + o.o_score, nq * k * 4);
  memcpy(out->cont_len, h_out + o.o_len, nq * k * 4);
  memcpy(out->cont_tok, h_out + o.o_tok, nq * k * L * 4);
  memcpy(out->fired, h_out + o.o_fired, nq * 4);
  return OILBIRD_OK;
}

static int host_step(oilbird_pool_t* p, bool do_append, const void* states, const int32_t* tokens,
                     int64_t n, uint64_t tag, uint32_t flags, const void* q, int32_t nq,
                     const oilbird_query_params* pr, const oilbird_query_out* out, void* stream) {
  if (!out_ok(out, true)) return OILBIRD_EINVAL;
  // (a slot and a staging block of their own: steps may be in flight beside this call)
  int rc = host_begin(p, do_append, states, tokens, n, tag, flags, q, nq, pr, kHostSlots, stream);
  if (rc) return rc;
  return host_end(p, kHostSlots, out);
}

int oilbird_pool_step_host_begin(oilbird_pool_t* p, const void* states, const int32_t* tokens,
                                 int64_t n, uint64_t tag, uint32_t flags, const void* q,
                                 int32_t nq, const oilbird_query_params* pr, int32_t slot,
                                 void* stream) {
  if (slot < 0 || slot >= kHostSlots) return OILBIRD_EINVAL;
  return host_begin(p, true, states, tokens, n, tag, flags, q, nq, pr, slot, stream);
}

int oilbird_pool_step_host_end(oilbird_pool_t* p, int32_t slot, const oilbird_query_out* out) {
  if (slot < 0 || slot >= kHostSlots) return OILBIRD_EINVAL;
  return host_end(p, slot, out);
}

int oilbird_pool_query_host(oilbird_pool_t* p, const void* q, int32_t nq,
                            const oilbird_query_params* pr, const oilbird_query_out* out,
                            void* stream) {
  return host_step(p, false, nullptr, nullptr, 0, 0, 0, q, nq, pr, out, stream);
}

int oilbird_pool_step_host(oilbird_pool_t* p, const void* states, const int32_t* tokens,
                           int64_t n, uint64_t tag, uint32_t flags, const void* q, int32_t nq,
                           const oilbird_query_params* pr, const oilbird_query_out* out,
                           void* stream) {
  return host_step(p, true, states, tokens, n, tag, flags, q, nq, pr, out, stream);
}

// ---- introspection ------------------------------------------------------------------

int oilbird_pool_status(oilbird_pool_t* p, oilbird_pool_stats* stats, void* stream) {
  if (!p) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  CU(cudaStreamSynchronize((cudaStream_t)stream));
  DeviceStats ds;
  CU(cudaMemcpy(&ds, p->stats, sizeof ds, cudaMemcpyDeviceToHost));
  if (stats) {
    stats->degenerate_rows = (int64_t)ds.degenerate_rows;
    stats->nonfinite_queries = (int64_t)ds.nonfinite_queries;
    stats->stalled = ds.stalled;
    stats->reserved = 0;
  }
  return ds.stalled ? OILBIRD_ESTALL : OILBIRD_OK;
}

int oilbird_pool_set_wait_limit(oilbird_pool_t* p, uint64_t limit_ns, void* stream) {
  if (!p) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  const unsigned long long v = limit_ns;
  // (pageable source: the call returns once the value has been staged)
  CU(cudaMemcpyAsync(&p->stats->wait_limit_ns, &v, sizeof v, cudaMemcpyHostToDevice,
                     (cudaStream_t)stream));
  return OILBIRD_OK;
}

int oilbird_pool_stall_selftest(oilbird_pool_t* p, void* stream) {
  if (!p) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  cudaError_t e = launch_stall_selftest(p->fuse_ready, p->stats, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "self-test kernel launch");
  p->launches += 1;
  return OILBIRD_OK;
}

int oilbird_pool_check_guards(oilbird_pool_t* p, void* stream) {
  if (!p) return OILBIRD_EINVAL;
  if (!p->r.guards) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  CU(cudaStreamSynchronize((cudaStream_t)stream));
  std::vector<unsigned char> buf;
  for (int g = 0; g < p->lay.n_guards; ++g) {
    const size_t n = p->lay.g_hi[g] - p->lay.g_lo[g];
    buf.resize(n);
    CU(cudaMemcpy(buf.data(), p->base + p->lay.g_lo[g], n, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < n; ++i) {
      if (buf[i] != kGuardByte) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "guard zone behind '%s' overwritten at byte %zu",
                 p->lay.g_name[g], i);
        return OILBIRD_EGUARD;
      }
    }
  }
  return OILBIRD_OK;
}

int oilbird_pool_read_rows(oilbird_pool_t* p, int64_t row0, int64_t n, void* keys,
                           int32_t* tokens, int32_t* trace_ids) {
  if (!p || row0 < 0 || n < 0 || row0 + n > p->n_rows) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  CU(cudaDeviceSynchronize());
  if (keys && p->r.e4m3) return OILBIRD_EINVAL;       // 8-bit pool: oilbird_pool_read_codes
  if (n == 0) return OILBIRD_OK;
  if (keys)
    CU(cudaMemcpy(keys, p->keys + (size_t)row0 * p->r.d, (size_t)n * p->r.d * 2,
                  cudaMemcpyDeviceToHost));
  if (tokens) CU(cudaMemcpy(tokens, p->tok + row0, (size_t)n * 4, cudaMemcpyDeviceToHost));
  if (trace_ids)
    CU(cudaMemcpy(trace_ids, p->trace_id + row0, (size_t)n * 4, cudaMemcpyDeviceToHost));
  return OILBIRD_OK;
}

int oilbird_pool_read_codes(oilbird_pool_t* p, int64_t row0, int64_t n, uint8_t* codes,
                            float* scales) {
  if (!p || !p->r.e4m3 || row0 < 0 || n < 0 || row0 + n > p->n_rows) return OILBIRD_EINVAL;
  CU(cudaSetDevice(p->device));
  CU(cudaDeviceSynchronize());
  if (n == 0) return OILBIRD_OK;
  if (codes)
    CU(cudaMemcpy(codes, p->codes + (size_t)row0 * p->r.d, (size_t)n * p->r.d,
                  cudaMemcpyDeviceToHost));
  if (scales) CU(cudaMemcpy(scales, p->scales + row0, (size_t)n * 4, cudaMemcpyDeviceToHost));
  return OILBIRD_OK;
}

int32_t oilbird_pool_read_traces(const oilbird_pool_t* p, int64_t* start, int64_t* end,
                                 uint64_t* tag, int32_t max_traces) {
  if (!p) return 0;
  int32_t n = (int32_t)p->t_start.size();
  int32_t m = n < max_traces ? n : max_traces;
  for (int32_t i = 0; i < m; ++i) {
    if (start) start[i] = p->t_start[i];
    if (end) end[i] = p->t_end[i];
    if (tag) tag[i] = p->t_tag[i];
  }
  return n;
}

int oilbird_pool_profile(oilbird_pool_t* p, int32_t enable) {
  if (!p) return OILBIRD_EINVAL;
  if (enable) {
    // all events now, none on the query path
    CU(cudaSetDevice(p->device));
    while ((int)p->ev.size() < 2 * kMaxProfile) {
      cudaEvent_t ne;
      CU(cudaEventCreate(&ne));
      p->ev.push_back(ne);
    }
  }
  p->profile = enable != 0;
  return OILBIRD_OK;
}

int32_t oilbird_pool_profile_read(oilbird_pool_t* p, float* scan_ms, int32_t max_n) {
  if (!p) return 0;
  cudaSetDevice(p->device);
  int32_t n = p->ev_used / 2, w = 0;
  for (int32_t i = 0; i < n; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(p->ev[2 * i + 1]) != cudaSuccess) break;
    if (cudaEventElapsedTime(&ms, p->ev[2 * i], p->ev[2 * i + 1]) != cudaSuccess) break;
    if (scan_ms && w < max_n) scan_ms[w++] = ms;
  }
  p->ev_used = 0;
  return w;
}

}  // extern "C"
