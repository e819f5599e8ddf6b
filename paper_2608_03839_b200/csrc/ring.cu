// Recycled pool: ring buffer of rejected-branch records and its lookup.
//
// Paper Section 4 "(i b) Recycling" and Algorithm 1's recycled-pool line: records keyed
// by (state in front of a rejected draft token, that token), valued by the continuation
// the model endorsed; a lookup returns at most m records with an equal anchor token and
// a cosine of at least `floor`, best first.
//
// Append is the hot side (every verification pass stores its rejected nodes): one CTA per
// record normalises the state into the slot it overwrites.  The lookup first compares
// anchor tokens (4 bytes per slot, coalesced) and streams the 16-byte key chunks of the
// matching slots only, so its traffic is capacity*4 + matches*d*2 bytes instead of the
// whole ring; each warp keeps its best records in a sorted register list, CTAs publish
// one list each, and the last CTA of a query to finish merges them and copies the
// continuations out (no second launch).  oilbird_ring_step also stores the records of a
// verification pass inside the same launch.
#include <math.h>
#include <stdio.h>

#include <new>

#include "common.cuh"
#include "internal.h"
#include "normalize.cuh"

namespace oilbird {

constexpr int kRingThreads = kNormThreads;
constexpr int kRingWarps = kRingThreads / 32;
constexpr int kRingList = 32;          // candidates per published list (>= OILBIRD_RING_MAX_M)

__global__ void __launch_bounds__(kRingThreads)
ring_append_kernel(const uint16_t* __restrict__ states, const int32_t* __restrict__ anchors,
                   const int32_t* __restrict__ rollouts, int64_t n, int d, int R, int64_t start,
                   int64_t cap, uint16_t* __restrict__ keys, int32_t* __restrict__ anchor,
                   int32_t* __restrict__ rollout) {
  pdl_enter();   // an earlier lookup may still be reading the slots this append overwrites
  for (int64_t r = blockIdx.x; r < n; r += gridDim.x) {
    const int64_t slot = (start + r) % cap;
    normalize_row(states + r * d, keys + slot * d, d);
    if (threadIdx.x == 0) anchor[slot] = anchors[r];
    if (threadIdx.x < R) rollout[slot * R + threadIdx.x] = rollouts[r * R + threadIdx.x];
  }
}

// The records of a step that the lookup's own kernel stores before it scans (oilbird_ring_step):
// n = 0 for a plain lookup.
struct RingFused {
  const uint16_t* states;
  const int32_t *anchors, *rollouts;
  int32_t* rollout;              // the ring's continuations (written here, read by the merge)
  int n, R;
  int64_t start, cap;            // record r goes to slot (start + r) % cap
  unsigned long long* ready;     // += 1 per stored record
  unsigned long long target;     // *ready once all n are in
};

// grid (slices, nq): CTA (s, q) scans slots [lo, hi) of the ring for query q.  With fused
// records the CTAs first store them, one record per CTA and round (all CTAs of the launch are
// resident together: at most two per SM are launched), and a warp whose 32 slots include a
// slot written by this launch waits, bounded, until all of them are in and reads those
// slots' anchors and keys through L2.
__global__ void __launch_bounds__(kRingThreads, 2)
ring_scan_kernel(uint16_t* __restrict__ keys, int32_t* __restrict__ anchor,
                 int64_t n_slots, int d, const uint16_t* __restrict__ q_raw,
                 const int32_t* __restrict__ q_anchor, int nq, int m, float floor_s,
                 u64* __restrict__ partial, int32_t* __restrict__ q_valid, DeviceStats* stats,
                 RingFused fa, unsigned* __restrict__ done, const int32_t* __restrict__ rollout,
                 int R, oilbird_ring_out out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_chunks = d >> 3;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                           // [n_chunks]
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)d * 2);          // [warps][32]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = blockIdx.y;
  pdl_enter();
  if (fa.n > 0) {
    const int n_blocks = gridDim.x * gridDim.y, b = blockIdx.y * gridDim.x + blockIdx.x;
    for (int r = b; r < fa.n; r += n_blocks) {
      const int64_t slot = (fa.start + r) % fa.cap;
      normalize_row(fa.states + (size_t)r * d, keys + slot * d, d);
      if (threadIdx.x == 0) anchor[slot] = fa.anchors[r];
      if (threadIdx.x < fa.R) fa.rollout[slot * fa.R + threadIdx.x] = fa.rollouts[(size_t)r * fa.R + threadIdx.x];
      __threadfence();                   // this thread's part of the record, before the count
      __syncthreads();
      if (threadIdx.x == 0) {
        __threadfence();                 // cumulative: the whole CTA's record
        atomicAdd(fa.ready, 1ull);
      }
    }
  }
  bool fresh_ok = fa.n == 0;             // this warp has seen the step's records arrive
  // slots written by this launch: [f0, f0 + n) modulo the ring's capacity
  const int64_t f0 = fa.n > 0 ? fa.start % fa.cap : 0;
  auto fresh = [&](int64_t slot) {
    if (fa.n == 0) return false;
    const int64_t off = slot >= f0 ? slot - f0 : slot + fa.cap - f0;
    return off < fa.n;
  };
  const int code = normalize_row<false>(q_raw + (size_t)q * d, reinterpret_cast<uint16_t*>(qs), d);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    q_valid[q] = code == kRowNonFinite ? 0 : 1;
    if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
  }
  __syncthreads();
  const int xq = q_anchor[q];
  const int64_t lo = n_slots * blockIdx.x / gridDim.x, hi = n_slots * (blockIdx.x + 1) / gridDim.x;
  const uint4* keys4 = reinterpret_cast<const uint4*>(keys);

  u64 top[1] = {0};
  u64 kth = 0;
  for (int64_t base = lo + warp * 32; base < hi; base += kRingWarps * 32) {
    const int64_t slot = base + lane;
    const bool mine_fresh = slot < hi && fresh(slot);
    const bool any_fresh = __any_sync(0xffffffffu, mine_fresh);
    if (any_fresh && !fresh_ok) {
      wait_fused_rows(fa.ready, fa.target, stats);
      fresh_ok = true;
    }
    const int a_slot = slot < hi ? (mine_fresh ? __ldcg(&anchor[slot]) : anchor[slot]) : 0;
    const bool hit = slot < hi && a_slot == xq;                // anchor token must be equal
    unsigned mask = __ballot_sync(0xffffffffu, hit);
    const unsigned fresh_mask = __ballot_sync(0xffffffffu, mine_fresh);
    while (mask) {
      const int src = __ffs(mask) - 1;
      mask &= mask - 1;
      const int64_t s_row = base + src;
      const uint4* rowp = keys4 + (size_t)s_row * n_chunks;
      const bool row_fresh = (fresh_mask >> src) & 1u;           // warp-uniform
      float acc = 0.f;
#pragma unroll 4
      for (int c = lane; c < n_chunks; c += 32) {
        const uint4 kv = row_fresh ? ld_cg16(rowp + c) : ld_stream16(rowp + c);
        const uint4 qv = qs[c];
        acc = fmaf(bf16_lo(kv.x), bf16_lo(qv.x), acc);
        acc = fmaf(bf16_hi(kv.x), bf16_hi(qv.x), acc);
        acc = fmaf(bf16_lo(kv.y), bf16_lo(qv.y), acc);
        acc = fmaf(bf16_hi(kv.y), bf16_hi(qv.y), acc);
        acc = fmaf(bf16_lo(kv.z), bf16_lo(qv.z), acc);
        acc = fmaf(bf16_hi(kv.z), bf16_hi(qv.z), acc);
        acc = fmaf(bf16_lo(kv.w), bf16_lo(qv.w), acc);
        acc = fmaf(bf16_hi(kv.w), bf16_hi(qv.w), acc);
      }
      const float s = warp_sum(acc);
      if (s >= floor_s) {                                      // cosine floor, per record
        const u64 key = pack_candidate(s, (uint32_t)s_row);
        if (key > kth) {
          warp_sorted_insert<1>(top, key, lane);
          kth = warp_list_get<1>(top, m - 1);
        }
      }
    }
  }
  block_merge_desc<1>(top, scratch, kRingWarps);
  if (threadIdx.x < 32) __stcg(&partial[((size_t)blockIdx.x * nq + q) * kRingList + lane], top[0]);

  // The last block of a query to get here merges the blocks' lists and writes the answer:
  // no launch of its own for that (a lookup moves under a megabyte and is bound by launch
  // latency; as a second kernel the merge cost a pass 5-6 us).
  __shared__ int s_last;
  __shared__ u64 s_best[kRingList];
  __threadfence();                       // this block's list (and any record it stored)
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned prev = atomicAdd(&done[q], 1u);
    s_last = prev == gridDim.x - 1;
    if (s_last) done[q] = 0;             // everybody has arrived: ready for the next launch
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();                       // the other blocks' lists, published before their arrival
  u64 v[1] = {0};
  if (code != kRowNonFinite) {           // a NaN/Inf query finds nothing
    // most blocks found nothing (a few dozen records match among hundreds of blocks): a warp
    // first looks at the heads of 32 lists at once, then fetches the lists that hold
    // something four at a time
    for (int l0 = warp * 32; l0 < (int)gridDim.x; l0 += kRingWarps * 32) {
      const int l = l0 + lane;
      const u64 head = l < (int)gridDim.x ? __ldcg(&partial[((size_t)l * nq + q) * kRingList]) : 0;
      unsigned live = __ballot_sync(0xffffffffu, head != 0);
      while (live) {
        u64 b[4][1];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int src = live ? __ffs(live) - 1 : -1;
          if (live) live &= live - 1;
          b[u][0] = src >= 0 ? __ldcg(&partial[((size_t)(l0 + src) * nq + q) * kRingList + lane]) : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) warp_merge_desc<1>(v, b[u], lane);
      }
    }
  }
  block_merge_desc<1>(v, scratch, kRingWarps);
  if (threadIdx.x < 32) s_best[lane] = v[0];
  __syncthreads();
  if (threadIdx.x == 0) {
    int c = 0;
    while (c < m && s_best[c] != 0) ++c;
    out.count[q] = c;
  }
  for (int j = threadIdx.x; j < m; j += kRingThreads) {
    const u64 key = s_best[j];
    out.slot[(size_t)q * m + j] = key ? candidate_row(key) : -1;
    out.score[(size_t)q * m + j] = key ? candidate_score(key) : -INFINITY;
    // stored continuation up to its first negative entry, -1 behind it (through L2: the
    // record may have been stored by another block of this launch)
    int len = 0;
    bool open = key != 0;
    for (int t = 0; t < R; ++t) {
      int tok = open ? __ldcg(&rollout[(size_t)candidate_row(key) * R + t]) : -1;
      if (tok < 0) open = false;
      out.rollout[((size_t)q * m + j) * R + t] = open ? tok : -1;
      if (open) ++len;
    }
    out.rollout_len[(size_t)q * m + j] = len;
  }
}

cudaError_t preload_ring_kernels() {
  cudaError_t e;
  if ((e = preload_kernel(ring_append_kernel)) != cudaSuccess) return e;
  return preload_kernel(ring_scan_kernel, true);
}

}  // namespace oilbird

using namespace oilbird;

static thread_local char g_ring_err[256] = "";
static int ring_fail(cudaError_t e, const char* what) {
  snprintf(g_ring_err, sizeof g_ring_err, "%s: %s", what, cudaGetErrorString(e));
  return e == cudaErrorMemoryAllocation ? OILBIRD_ENOMEM : OILBIRD_ECUDA;
}
#define RCU(call)                                         \
  do {                                                    \
    cudaError_t e_ = (call);                              \
    if (e_ != cudaSuccess) return ring_fail(e_, #call);   \
  } while (0)

struct oilbird_ring {
  int32_t d, R, device, num_sms, max_lists;
  int64_t cap, total;
  uint16_t* keys;
  int32_t *anchor, *rollout, *q_valid;
  unsigned long long* partial;
  DeviceStats* stats;
  unsigned* done;                  // per query: blocks of the running lookup that have finished
  unsigned long long* ready;       // records stored by lookups that append (device counter) ...
  unsigned long long ready_target; // ... and the host's count of them (enqueue time)
  unsigned char* base;
};

extern "C" {

int oilbird_ring_create(oilbird_ring_t** out, const oilbird_ring_config* cfg) {
  if (!out || !cfg) return OILBIRD_EINVAL;
  *out = nullptr;
  if (cfg->d < 8 || cfg->d > 16384 || cfg->d % 8 != 0 || cfg->capacity < 1 ||
      cfg->capacity > 2147483000LL || cfg->max_rollout < 0 ||
      cfg->max_rollout > OILBIRD_RING_MAX_ROLLOUT)
    return OILBIRD_EINVAL;
  int n_dev = 0;
  RCU(cudaGetDeviceCount(&n_dev));
  if (cfg->device < 0 || cfg->device >= n_dev) return OILBIRD_EINVAL;
  RCU(cudaSetDevice(cfg->device));
  RCU(preload_all_kernels());      // before anything of the library is launched on this device
  int sms = 0;
  RCU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device));
  oilbird_ring* r = new (std::nothrow) oilbird_ring();
  if (!r) return OILBIRD_ENOMEM;
  r->d = cfg->d; r->R = cfg->max_rollout ? cfg->max_rollout : 6; r->device = cfg->device;
  r->num_sms = sms; r->max_lists = 2 * sms; r->cap = cfg->capacity; r->total = 0;
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  const size_t o_keys = 0, o_anchor = up((size_t)r->cap * r->d * 2),
               o_roll = o_anchor + up((size_t)r->cap * 4),
               o_valid = o_roll + up((size_t)r->cap * r->R * 4),
               o_part = o_valid + up((size_t)OILBIRD_RING_MAX_NQ * 4),
               o_stats = o_part + up((size_t)r->max_lists * OILBIRD_RING_MAX_NQ * kRingList * 8),
               o_ready = o_stats + up(sizeof(DeviceStats)), o_done = o_ready + 256,
               total = o_done + up((size_t)OILBIRD_RING_MAX_NQ * 4);
  void* mem = nullptr;
  cudaError_t e = cudaMalloc(&mem, total);
  if (e != cudaSuccess) { delete r; return ring_fail(e, "cudaMalloc(ring)"); }
  r->base = (unsigned char*)mem;
  r->keys = (uint16_t*)(r->base + o_keys);
  r->anchor = (int32_t*)(r->base + o_anchor);
  r->rollout = (int32_t*)(r->base + o_roll);
  r->q_valid = (int32_t*)(r->base + o_valid);
  r->partial = (unsigned long long*)(r->base + o_part);
  r->stats = (DeviceStats*)(r->base + o_stats);
  r->ready = (unsigned long long*)(r->base + o_ready);
  r->done = (unsigned*)(r->base + o_done);
  r->ready_target = 0;
  e = cudaMemset(r->stats, 0, total - o_stats);               // counters, fused-store and arrival counters
  if (e != cudaSuccess) { cudaFree(mem); delete r; return ring_fail(e, "cudaMemset"); }
  *out = r;
  return OILBIRD_OK;
}

int oilbird_ring_destroy(oilbird_ring_t* r) {
  if (!r) return OILBIRD_EINVAL;
  cudaSetDevice(r->device);
  cudaDeviceSynchronize();
  cudaFree(r->base);
  delete r;
  return OILBIRD_OK;
}

int oilbird_ring_reset(oilbird_ring_t* r, void* stream) {
  if (!r) return OILBIRD_EINVAL;
  RCU(cudaSetDevice(r->device));
  RCU(cudaMemsetAsync(r->stats, 0, sizeof(DeviceStats), (cudaStream_t)stream));
  r->total = 0;
  return OILBIRD_OK;
}

int64_t oilbird_ring_size(const oilbird_ring_t* r) {
  return r ? (r->total < r->cap ? r->total : r->cap) : 0;
}
int64_t oilbird_ring_total(const oilbird_ring_t* r) { return r ? r->total : 0; }

int oilbird_ring_append(oilbird_ring_t* r, const void* states, const int32_t* anchors,
                        const int32_t* rollouts, int64_t n, void* stream) {
  if (!r || n < 0 || (n > 0 && (!states || !anchors || !rollouts))) return OILBIRD_EINVAL;
  if (n == 0) return OILBIRD_OK;
  RCU(cudaSetDevice(r->device));
  // more records than slots: only the last `capacity` of them survive
  const int64_t skip = n > r->cap ? n - r->cap : 0;
  const int64_t m = n - skip;
  const int64_t grid = m > 65535 * 8 ? 65535 * 8 : m;
  cudaError_t e = launch_pdl(ring_append_kernel, dim3((unsigned)grid), dim3(kRingThreads), 0,
                             (cudaStream_t)stream,
                             (const uint16_t*)states + (size_t)skip * r->d, anchors + skip,
                             rollouts + (size_t)skip * r->R, m, r->d, r->R, r->total + skip, r->cap,
                             r->keys, r->anchor, r->rollout);
  if (e != cudaSuccess) return ring_fail(e, "ring append launch");
  r->total += n;
  return OILBIRD_OK;
}

// Lookup, optionally with the records of a step stored by the scan kernel itself.
static int ring_query_impl(oilbird_ring_t* r, const void* q, const int32_t* q_anchor, int32_t nq,
                           int32_t m, float floor_s, const oilbird_ring_out* out, void* stream,
                           const void* states, const int32_t* anchors, const int32_t* rollouts,
                           int64_t n) {
  if (!r || !q || !q_anchor || !out || !out->slot || !out->score || !out->count ||
      !out->rollout || !out->rollout_len)
    return OILBIRD_EINVAL;
  if (nq < 1 || nq > OILBIRD_RING_MAX_NQ || m < 1 || m > OILBIRD_RING_MAX_M || isnan(floor_s))
    return OILBIRD_EINVAL;
  RCU(cudaSetDevice(r->device));
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t total_after = r->total + n;
  const int64_t n_slots = total_after < r->cap ? total_after : r->cap;
  // at least 256 slots per CTA, at most two CTAs per SM
  int64_t want = (n_slots + 255) / 256;
  int slices = (int)(want < 1 ? 1 : (want > r->max_lists ? r->max_lists : want));
  RingFused fa = {};
  if (n > 0) {
    // the scan's own blocks store the records: they must all be resident together, because
    // scanning warps wait for the storing ones (else: a launch of its own for the append)
    if ((int64_t)slices * nq > 2 * r->num_sms || n > r->cap) {
      int rc = oilbird_ring_append(r, states, anchors, rollouts, n, stream);
      if (rc) return rc;
      return ring_query_impl(r, q, q_anchor, nq, m, floor_s, out, stream, nullptr, nullptr, nullptr, 0);
    }
    fa.states = (const uint16_t*)states; fa.anchors = anchors; fa.rollouts = rollouts;
    fa.rollout = r->rollout; fa.n = (int)n; fa.R = r->R; fa.start = r->total; fa.cap = r->cap;
    fa.ready = r->ready; fa.target = r->ready_target + (unsigned long long)n;
  }
  const size_t smem = (size_t)r->d * 2 + (size_t)kRingWarps * kRingList * sizeof(u64);
  cudaError_t e = launch_pdl(ring_scan_kernel, dim3(slices, nq), dim3(kRingThreads), smem, st,
                             r->keys, r->anchor, n_slots, r->d, (const uint16_t*)q, q_anchor, nq, m,
                             floor_s, r->partial, r->q_valid, r->stats, fa, r->done,
                             (const int32_t*)r->rollout, r->R, *out);
  if (e != cudaSuccess) return ring_fail(e, "ring scan launch");
  if (n > 0) {
    r->total = total_after;
    r->ready_target = fa.target;
  }
  return OILBIRD_OK;
}

int oilbird_ring_query(oilbird_ring_t* r, const void* q, const int32_t* q_anchor, int32_t nq,
                       int32_t m, float floor_s, const oilbird_ring_out* out, void* stream) {
  return ring_query_impl(r, q, q_anchor, nq, m, floor_s, out, stream, nullptr, nullptr, nullptr, 0);
}

int oilbird_ring_step(oilbird_ring_t* r, const void* states, const int32_t* anchors,
                      const int32_t* rollouts, int64_t n, const void* q, const int32_t* q_anchor,
                      int32_t nq, int32_t m, float floor_s, const oilbird_ring_out* out,
                      void* stream) {
  if (n < 0 || (n > 0 && (!states || !anchors || !rollouts))) return OILBIRD_EINVAL;
  return ring_query_impl(r, q, q_anchor, nq, m, floor_s, out, stream, states, anchors, rollouts, n);
}

int oilbird_ring_read(oilbird_ring_t* r, void* keys, int32_t* anchors, int32_t* rollouts) {
  if (!r) return OILBIRD_EINVAL;
  RCU(cudaSetDevice(r->device));
  RCU(cudaDeviceSynchronize());
  if (keys) RCU(cudaMemcpy(keys, r->keys, (size_t)r->cap * r->d * 2, cudaMemcpyDeviceToHost));
  if (anchors) RCU(cudaMemcpy(anchors, r->anchor, (size_t)r->cap * 4, cudaMemcpyDeviceToHost));
  if (rollouts)
    RCU(cudaMemcpy(rollouts, r->rollout, (size_t)r->cap * r->R * 4, cudaMemcpyDeviceToHost));
  return OILBIRD_OK;
}

const char* oilbird_ring_last_error(void) { return g_ring_err; }

}  // extern "C"
