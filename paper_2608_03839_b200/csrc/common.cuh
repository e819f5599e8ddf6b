// Device-side helpers shared by the pool's kernels: candidate packing and warp-level
// sorted candidate lists (bitonic sort / merge, shuffle insertion).  Nothing here is visible outside the CUDA library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "internal.h"

namespace oilbird {

typedef unsigned long long u64;

// ---------------------------------------------------------------- candidates ---
// A candidate (score, row) is packed into one 64-bit key whose unsigned order is the
// order of Eq. 2 plus the tie rule: higher score first, lower row first.  The high
// word is the usual order-preserving map of an IEEE float, the low word is ~row.
// Key 0 never occurs for a real candidate and marks an empty slot.

__device__ __forceinline__ u64 pack_candidate(float s, uint32_t row) {
  s += 0.0f;                                   // -0.0 -> +0.0 so the two compare equal
  uint32_t b = __float_as_uint(s);
  b = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return ((u64)b << 32) | (u64)(~row);
}
__device__ __forceinline__ float candidate_score(u64 key) {
  uint32_t b = (uint32_t)(key >> 32);
  b = (b & 0x80000000u) ? (b & 0x7fffffffu) : ~b;
  return __uint_as_float(b);
}
__device__ __forceinline__ int32_t candidate_row(u64 key) { return (int32_t)(~(uint32_t)key); }

// ------------------------------------------------------------------- bf16 ------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// round-to-nearest-even float -> bf16 bits (finite inputs)
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint32_t u = __float_as_uint(f);
  u += 0x7fffu + ((u >> 16) & 1u);
  return u >> 16;
}

// streaming 16-byte load: read-only path, do not keep in L1
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// coherent 16-byte load (L2): for rows that another CTA of the same launch has just written
__device__ __forceinline__ uint4 ld_cg16(const void* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// The pool's limit for device-side waits (two seconds unless the caller set another).
__device__ __forceinline__ unsigned long long wait_limit_ns(const DeviceStats* stats) {
  const unsigned long long v = *reinterpret_cast<const volatile unsigned long long*>(&stats->wait_limit_ns);
  return v ? v : kDefaultWaitNs;
}

// A scan whose first CTAs append the step's rows: wait until all of them are in (every
// appending CTA adds one to *ready after its row).  Bounded: after the pool's wait limit the
// `stalled` flag is raised and the caller carries on (the status call reports it).
__device__ __forceinline__ void wait_fused_rows(const unsigned long long* ready,
                                                unsigned long long target, DeviceStats* stats) {
  unsigned long long t0 = 0, limit = 0;
  for (uint32_t spin = 0; ld_acquire_u64(ready) < target; ++spin) {
    if (spin == 0) {
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
      limit = wait_limit_ns(stats);
    }
    if ((spin & 15u) == 15u) {
      unsigned long long t1;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
      if (t1 - t0 > limit) { atomicExch(&stats->stalled, 1); break; }
    }
    __nanosleep(64);
  }
}
__device__ __forceinline__ void wait_fused_rows(const FusedAppend& fa, DeviceStats* stats) {
  wait_fused_rows(fa.ready, fa.target, stats);
}
// Wait until another CTA of this launch has raised a flag word (acquire).  Bounded in the same
// way: false after the pool's wait limit, with `stalled` raised.
__device__ __forceinline__ bool wait_flag_u32(const unsigned* flag, DeviceStats* stats) {
  unsigned long long t0 = 0, limit = 0;
  for (uint32_t spin = 0;; ++spin) {
    unsigned r;
    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(r) : "l"(flag) : "memory");
    if (r != 0) return true;
    if (spin == 0) {
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
      limit = wait_limit_ns(stats);
    }
    if ((spin & 15u) == 15u) {
      unsigned long long t1;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
      if (t1 - t0 > limit) { atomicExch(&stats->stalled, 1); return false; }
    }
    __nanosleep(64);
  }
}

// ------------------------------------------------- scoring rows (CUDA cores) ---
constexpr int kRowsPerIter = 4;   // rows a warp scores together (shares each query load)
// Dot products of kRowsPerIter rows with the QT queries in shared memory; kFresh selects
// the coherent load for rows written during this launch.
template <int QT, bool kFresh>
__device__ __forceinline__ void score_rows(const uint4* const (&rowp)[kRowsPerIter], const uint4* qs,
                                           int n_chunks, int lane,
                                           float (&acc)[kRowsPerIter][QT]) {
#pragma unroll 2
  for (int c = lane; c < n_chunks; c += 32) {
    uint4 kv[kRowsPerIter];
#pragma unroll
    for (int r = 0; r < kRowsPerIter; ++r)
      kv[r] = kFresh ? ld_cg16(rowp[r] + c) : ld_stream16(rowp[r] + c);
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      const uint4 qv = qs[q * n_chunks + c];
      const float q0f = bf16_lo(qv.x), q1f = bf16_hi(qv.x), q2f = bf16_lo(qv.y),
                  q3f = bf16_hi(qv.y), q4f = bf16_lo(qv.z), q5f = bf16_hi(qv.z),
                  q6f = bf16_lo(qv.w), q7f = bf16_hi(qv.w);
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r) {
        float a = acc[r][q];
        a = fmaf(bf16_lo(kv[r].x), q0f, a);
        a = fmaf(bf16_hi(kv[r].x), q1f, a);
        a = fmaf(bf16_lo(kv[r].y), q2f, a);
        a = fmaf(bf16_hi(kv[r].y), q3f, a);
        a = fmaf(bf16_lo(kv[r].z), q4f, a);
        a = fmaf(bf16_hi(kv[r].z), q5f, a);
        a = fmaf(bf16_lo(kv[r].w), q6f, a);
        a = fmaf(bf16_hi(kv[r].w), q7f, a);
        acc[r][q] = a;
      }
    }
  }
}

// ---------------------------------------------------- programmatic launch ------
// The kernels of a step may be launched with programmatic stream serialization (see
// launch_pdl in internal.h): a kernel's blocks can then be scheduled, and run their set-up,
// while the previous kernel of the stream is still working, which hides the launch latency
// between the three or four kernels of a step.  pdl_enter() must come before the first
// access to anything an earlier kernel wrote: it waits for that kernel to finish and its
// writes to be visible, and only then lets the NEXT kernel of the stream be scheduled.
// Releasing the successor after the wait, not before it, bounds the chain: at most two
// grids are on the GPU at any time, the one that works and the one that is set up and
// waiting for it; a kernel never sits behind a predecessor that is itself still waiting.
// Both instructions are no-ops for a plain launch.
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ------------------------------------------------------------------ warp ops ---
__device__ __forceinline__ u64 shfl_xor_u64(u64 v, int m) {
  uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)v, m);
  uint32_t hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(v >> 32), m);
  return ((u64)hi << 32) | lo;
}
__device__ __forceinline__ u64 warp_min_u64(u64 v) {
#pragma unroll
  for (int m = 16; m; m >>= 1) { u64 o = shfl_xor_u64(v, m); v = o < v ? o : v; }
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int m = 16; m; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
  return v;
}

// --------------------------------------------------- warp-level sorted lists ---
// A list of K = 32*E packed candidates lives in the registers of one warp: element i is
// v[i / 32] of lane i % 32.  Both routines are bitonic networks; strides >= 32 pair two
// registers of the same lane, strides < 32 are xor-shuffles.

template <int E>
__device__ __forceinline__ void warp_bitonic_stage(u64 (&v)[E], int lane, int size, int stride) {
  if (stride >= 32) {
    const int rs = stride >> 5;
#pragma unroll
    for (int r = 0; r < E; ++r) {
      if ((r & rs) == 0) {
        const int i = r * 32 + lane;
        const bool desc = (i & size) == 0;
        u64 a = v[r], b = v[r | rs];
        const bool sw = desc ? (a < b) : (a > b);
        v[r] = sw ? b : a;
        v[r | rs] = sw ? a : b;
      }
    }
  } else {
#pragma unroll
    for (int r = 0; r < E; ++r) {
      const int i = r * 32 + lane;
      const u64 o = shfl_xor_u64(v[r], stride);
      const bool lower = (i & stride) == 0;
      const bool desc = (i & size) == 0;
      const bool keep_max = lower == desc;
      const u64 mx = v[r] > o ? v[r] : o, mn = v[r] > o ? o : v[r];
      v[r] = keep_max ? mx : mn;
    }
  }
}

// Sort the K elements descending.
template <int E>
__device__ __forceinline__ void warp_sort_desc(u64 (&v)[E], int lane) {
#pragma unroll
  for (int size = 2; size <= 32 * E; size <<= 1)
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1)
      warp_bitonic_stage<E>(v, lane, size == 32 * E ? (1 << 30) : size, stride);
}

// a <- the K largest of (a U b), descending; a and b both sorted descending.
template <int E>
__device__ __forceinline__ void warp_merge_desc(u64 (&a)[E], const u64 (&b)[E], int lane) {
  // c[i] = max(a[i], b[K-1-i]) is bitonic and holds the K largest
#pragma unroll
  for (int r = 0; r < E; ++r) {
    const u64 src = b[E - 1 - r];
    const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)src, 31 - lane);
    const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)(src >> 32), 31 - lane);
    const u64 o = ((u64)hi << 32) | lo;
    a[r] = a[r] > o ? a[r] : o;
  }
#pragma unroll
  for (int stride = 16 * E; stride > 0; stride >>= 1)
    warp_bitonic_stage<E>(a, lane, 1 << 30, stride);
}

// The same networks over NB independent lists at once, list index innermost: a stage is a
// chain of a shuffle and half a dozen dependent ALU operations (~40 cycles), and the
// compiler keeps separate calls of the routines above one after the other, so NB lists
// sorted by NB calls take NB times as long; interleaved by hand they overlap (8 lists
// fill the issue slots).
template <int NB, int E>
__device__ __forceinline__ void warp_bitonic_stage_batch(u64 (&v)[NB][E], int lane, int size,
                                                         int stride) {
  if (stride >= 32) {
    const int rs = stride >> 5;
#pragma unroll
    for (int r = 0; r < E; ++r) {
      if ((r & rs) == 0) {
        const bool desc = ((r * 32 + lane) & size) == 0;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          const u64 x = v[b][r], y = v[b][r | rs];
          const bool sw = (x < y) == desc;
          v[b][r] = sw ? y : x;
          v[b][r | rs] = sw ? x : y;
        }
      }
    }
  } else {
#pragma unroll
    for (int r = 0; r < E; ++r) {
      const int i = r * 32 + lane;
      const bool keep_max = ((i & stride) == 0) == ((i & size) == 0);
      u64 o[NB];
#pragma unroll
      for (int b = 0; b < NB; ++b) o[b] = shfl_xor_u64(v[b][r], stride);
#pragma unroll
      for (int b = 0; b < NB; ++b) v[b][r] = ((v[b][r] > o[b]) == keep_max) ? v[b][r] : o[b];
    }
  }
}

template <int NB, int E>
__device__ __forceinline__ void warp_sort_desc_batch(u64 (&v)[NB][E], int lane) {
#pragma unroll
  for (int size = 2; size <= 32 * E; size <<= 1)
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1)
      warp_bitonic_stage_batch<NB, E>(v, lane, size == 32 * E ? (1 << 30) : size, stride);
}

// a[b] <- the K largest of (a[b] U c[b]) for every b; all lists sorted descending.
template <int NB, int E>
__device__ __forceinline__ void warp_merge_desc_batch(u64 (&a)[NB][E], const u64 (&c)[NB][E],
                                                      int lane) {
#pragma unroll
  for (int r = 0; r < E; ++r) {
    u64 o[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const u64 src = c[b][E - 1 - r];
      const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)src, 31 - lane);
      const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)(src >> 32), 31 - lane);
      o[b] = ((u64)hi << 32) | lo;
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) a[b][r] = a[b][r] > o[b] ? a[b][r] : o[b];
  }
#pragma unroll
  for (int stride = 16 * E; stride > 0; stride >>= 1)
    warp_bitonic_stage_batch<NB, E>(a, lane, 1 << 30, stride);
}

// Insert one candidate (the same key in every lane) into a descending register list,
// dropping the smallest element.  Branch-free (a key of 0, the empty slot, is a no-op in
// effect), so that several independent lists can be updated in interleaved straight-line
// code and hide each other's shuffle latency.  About a dozen instructions per 32 elements.
template <int E>
__device__ __forceinline__ void warp_sorted_insert(u64 (&v)[E], u64 key, int lane) {
#pragma unroll
  for (int r = 0; r < E; ++r) {
    const int pos = __popc(__ballot_sync(0xffffffffu, v[r] > key));   // elements that stay put
    const uint32_t ulo = __shfl_up_sync(0xffffffffu, (uint32_t)v[r], 1);
    const uint32_t uhi = __shfl_up_sync(0xffffffffu, (uint32_t)(v[r] >> 32), 1);
    const uint32_t clo = __shfl_sync(0xffffffffu, (uint32_t)v[r], 31);
    const uint32_t chi = __shfl_sync(0xffffffffu, (uint32_t)(v[r] >> 32), 31);
    const u64 up = ((u64)uhi << 32) | ulo;
    const u64 carry = ((u64)chi << 32) | clo;
    v[r] = lane < pos ? v[r] : (lane == pos ? key : up);              // pos == 32: unchanged
    key = pos < 32 ? carry : key;                                     // carried into the next row
  }
}

// Element i of a register list, broadcast to all lanes.
template <int E>
__device__ __forceinline__ u64 warp_list_get(const u64 (&v)[E], int i) {
  u64 x = v[0];
#pragma unroll
  for (int r = 1; r < E; ++r) x = (i >> 5) == r ? v[r] : x;
  const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)x, i & 31);
  const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)(x >> 32), i & 31);
  return ((u64)hi << 32) | lo;
}

// Merge the sorted register lists of all warps of the block into warp 0's registers.
// scratch: n_warps * 32 * E keys of shared memory.  All threads must call.
template <int E>
__device__ __forceinline__ void block_merge_desc(u64 (&v)[E], u64* scratch, int n_warps) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int half = (n_warps + 1) >> 1; n_warps > 1; n_warps = half, half = (n_warps + 1) >> 1) {
    __syncthreads();
    if (warp >= half && warp < n_warps) {
#pragma unroll
      for (int r = 0; r < E; ++r) scratch[(size_t)warp * 32 * E + r * 32 + lane] = v[r];
    }
    __syncthreads();
    if (warp + half < n_warps) {
      u64 b[E];
#pragma unroll
      for (int r = 0; r < E; ++r) b[r] = scratch[(size_t)(warp + half) * 32 * E + r * 32 + lane];
      warp_merge_desc<E>(v, b, lane);
    }
  }
}

// ------------------------------------------------------ final merge (one CTA) ---
constexpr int kMergeThreads = 1024;
constexpr int kMergeWarps = kMergeThreads / 32;

// Each warp folds its share of the scan's descending lists into a register-resident
// list of kk = 32*E candidates (bitonic merges), then the warps' lists are merged.
//
// All of this runs on one SM, where the merges are bound by shuffle throughput (32 warps
// folding ten lists each took 4 us), so lists that cannot matter are dropped first: a
// list's head is its best candidate; the k-th largest of the 32 warps' best heads is
// reached by k distinct lists, hence by k candidates, so no list whose head lies below
// it holds one of the k best.  For k <= 32 that leaves about one list per warp.
template <int E>
__device__ __forceinline__ void merge_lists(const u64* __restrict__ partial, int n_lists, int nq,
                                            int q, int k, u64* scratch, u64* s_best) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int KK = 32 * E;
  __shared__ u64 s_head[kMergeWarps];
  __shared__ u64 s_floor;
  u64 v[E];
#pragma unroll
  for (int r = 0; r < E; ++r) v[r] = 0;
  // many lists in flight per warp: the loads, not the merges, set the pace (with two CTAs
  // per SM a warp folds about ten lists, so one round of loads covers the common case)
  constexpr int PF = E == 1 ? 10 : (E == 2 ? 5 : 3);
  // (k == 0: the caller does not want the filter)
  const bool filter = k >= 1 && k <= kMergeWarps && n_lists <= kMergeWarps * PF;   // one round of loads
  u64 b[PF][E];
  if (filter) {
    u64 best = 0;
#pragma unroll
    for (int p = 0; p < PF; ++p) {
      const int l = warp + p * kMergeWarps;
      const u64* src = partial + ((size_t)(l < n_lists ? l : 0) * nq + q) * KK;
#pragma unroll
      for (int r = 0; r < E; ++r) b[p][r] = l < n_lists ? src[r * 32 + lane] : 0;
      best = b[p][0] > best ? b[p][0] : best;            // lane 0 holds the heads
    }
    if (lane == 0) s_head[warp] = best;
    __syncthreads();
    if (warp == 0) {
      u64 h[1] = {s_head[lane]};
      warp_sort_desc<1>(h, lane);
      const u64 f = warp_list_get<1>(h, k - 1);          // 0 while fewer than k lists exist
      if (lane == 0) s_floor = f;
    }
    __syncthreads();
    const u64 floor_key = s_floor;
#pragma unroll
    for (int p = 0; p < PF; ++p) {
      const u64 head = warp_list_get<E>(b[p], 0);
      if (head != 0 && head >= floor_key) warp_merge_desc<E>(v, b[p], lane);   // warp-uniform
    }
  } else {
    for (int l0 = warp; l0 < n_lists; l0 += kMergeWarps * PF) {
#pragma unroll
      for (int p = 0; p < PF; ++p) {
        const int l = l0 + p * kMergeWarps;
        const u64* src = partial + ((size_t)(l < n_lists ? l : 0) * nq + q) * KK;
#pragma unroll
        for (int r = 0; r < E; ++r) b[p][r] = l < n_lists ? src[r * 32 + lane] : 0;
      }
#pragma unroll
      for (int p = 0; p < PF; ++p)
        if (l0 + p * kMergeWarps < n_lists) warp_merge_desc<E>(v, b[p], lane);
    }
  }
  // the 32 warps' lists -> one: four warps fold eight lists each as a tree of interleaved
  // merges, then one warp folds those four (two barriers instead of ten)
#pragma unroll
  for (int r = 0; r < E; ++r) scratch[(size_t)warp * KK + r * 32 + lane] = v[r];
  __syncthreads();
  if (warp < 4) {
    // 8 -> 4 (two lists at a time: 1024 threads leave 64 registers each), 4 -> 2, 2 -> 1
    u64 m[4][E];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      u64 a[2][E], c[2][E];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int r = 0; r < E; ++r) {
          a[i][r] = scratch[(size_t)(warp * 8 + 2 * h + i) * KK + r * 32 + lane];
          c[i][r] = scratch[(size_t)(warp * 8 + 4 + 2 * h + i) * KK + r * 32 + lane];
        }
      warp_merge_desc_batch<2, E>(a, c, lane);
#pragma unroll
      for (int r = 0; r < E; ++r) { m[2 * h][r] = a[0][r]; m[2 * h + 1][r] = a[1][r]; }
    }
    u64 a2[2][E], c2[2][E];
#pragma unroll
    for (int r = 0; r < E; ++r) { a2[0][r] = m[0][r]; a2[1][r] = m[1][r]; c2[0][r] = m[2][r]; c2[1][r] = m[3][r]; }
    warp_merge_desc_batch<2, E>(a2, c2, lane);               // 4 -> 2
    warp_merge_desc<E>(a2[0], a2[1], lane);                  // 2 -> 1
#pragma unroll
    for (int r = 0; r < E; ++r) v[r] = a2[0][r];
  }
  __syncthreads();
  if (warp < 4) {
#pragma unroll
    for (int r = 0; r < E; ++r) scratch[(size_t)warp * KK + r * 32 + lane] = v[r];
  }
  __syncthreads();
  if (warp == 0) {
    u64 a[2][E], c[2][E];
#pragma unroll
    for (int r = 0; r < E; ++r) {
      a[0][r] = scratch[r * 32 + lane];
      a[1][r] = scratch[(size_t)KK + r * 32 + lane];
      c[0][r] = scratch[(size_t)2 * KK + r * 32 + lane];
      c[1][r] = scratch[(size_t)3 * KK + r * 32 + lane];
    }
    warp_merge_desc_batch<2, E>(a, c, lane);
    warp_merge_desc<E>(a[0], a[1], lane);
#pragma unroll
    for (int r = 0; r < E; ++r) s_best[r * 32 + lane] = a[0][r];
  }
  __syncthreads();
}

}  // namespace oilbird
