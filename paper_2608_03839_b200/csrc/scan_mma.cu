// K2b: warp-level tensor-core scan for small batches (8 or 16 queries per pass).
//
// Scoring line of Algorithm 1 (cosine of each query with every stored state) fused with the
// per-CTA part of Eq. 2's top-k, for the batch sizes between single-request decode and the
// large batches of the tcgen05 scan.  The tcgen05 scan needs whole 128-row tiles and a
// completed K loop before a score exists, which costs about 40 us per query call on pools of
// the paper's size (a few hundred MB); the CUDA-core scan runs out of issue slots beyond two
// queries (64 FMAs per 16 key bytes at eight).  Here the key stream is organised as in the
// CUDA-core scan (16 warps per SM, contiguous row split, 16-byte streaming loads straight
// into registers) and the arithmetic goes to mma.sync.m16n8k16 (bf16 in,
// fp32 accumulate): 16 rows x 8 queries x 32 elements cost two loads of keys, one shared
// memory load of queries and two MMAs per lane, so the kernel stays bound by the key stream.
//
// The reduction dimension may be walked in any order as long as keys and queries agree, so
// a lane's 16-byte load (eight consecutive elements of one row) feeds the k slots of two
// MMAs directly: lane (g, t) = (lane / 4, lane % 4) holds rows g and g + 8 of the group
// and elements 8 t .. 8 t + 7 of each 32-element block, and reads the same elements of
// query g from shared memory.  No shuffles, no staging of keys in shared memory.
//
// Each warp keeps one descending register list per query (Eq. 2); a group's 128 scores are
// tested against the lists' k-th entries and the few that pass are inserted one by one.  At
// the end warp w merges query w's lists; what leaves the CTA is one list per query, as in
// the other scans.
//
// Pools with 8-bit keys (E4M3 codes + one scale per row) run the same kernel with f16
// operands: a code is an f16 number exactly, the query is held as f16 scaled by 2^14.
#include <cuda_fp16.h>

#include "common.cuh"
#include "internal.h"
#include "normalize.cuh"
#include "quant8.cuh"

namespace oilbird {

constexpr int kMmaThreads = 512;   // one CTA of four quads of four warps per SM
constexpr int kMmaQ = 8;          // queries per pass = the N of the instruction
constexpr int kMmaRows = 16;      // rows per warp step = the M of the instruction
constexpr int kMmaDepth1 = 4;     // 32-element blocks per lane, row and step: 8-query form
constexpr int kMmaDepth2 = 2;     // 16-query form (its accumulators and lists need the registers)
constexpr int kMmaBatchInsert = 5; // candidates of a group and query from which they are merged in as a sorted vector
constexpr int kMmaPadBytes = 64;   // per query row in shared memory: keeps the 16-byte loads of
                                   // a quarter warp (two queries x four offsets) on distinct banks

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct BoolTrue { static constexpr bool value = true; };
struct BoolFalse { static constexpr bool value = false; };

// 16 bytes of a key: the read-only streaming path, or through L2 for rows that another CTA
// of this launch has just written
__device__ __forceinline__ uint4 ld_key16(const uint4* p, bool fresh) {
  return fresh ? ld_cg16(p) : ld_stream16(p);
}

// barrier among the four warps of a quad (ids 1 to 4; 0 is __syncthreads, 5 the quantising
// warps of an 8-bit step)
__device__ __forceinline__ void quad_bar(int id) {
  asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory");
}

// the same with f16 operands: pools with 8-bit keys (an E4M3 code is an f16 number exactly)
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                        uint32_t a3, uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two E4M3 codes (low 16 bits) -> f16x2, first code in the low half
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_codes) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)two_codes));
  return h2;
}
// queries of an 8-bit pool are held as f16 scaled by 2^14 (|q| <= 1 after normalisation; the
// scale keeps their small elements out of f16's subnormal range); the score is scaled back
constexpr float kFp8QueryScale = 16384.f;

// normalize_row done by one warp, with the numbers accumulated in the order of the block
// routine (lane l plays threads l, l + 32, ... l + 224 of a 256-thread block with one
// accumulator each), so that a query is normalised to the same bf16 vector on every path.
__device__ __forceinline__ int normalize_row_warp(const uint16_t* __restrict__ src,
                                                  uint16_t* __restrict__ dst, int d, int lane) {
  const int n_chunks = d >> 3;
  const uint4* src4 = reinterpret_cast<const uint4*>(src);
  uint4* dst4 = reinterpret_cast<uint4*>(dst);
  // Rows of normal finite numbers first (see normalize_row_regs: doubles built from the bits,
  // the same numbers as the conversions give): eight queries of three conversions per
  // element in every CTA would keep the conversion unit busy for microseconds.
  {
    double acc[kNormThreads / 32];
    uint32_t umin = 0xffffffffu;
#pragma unroll
    for (int v = 0; v < kNormThreads / 32; ++v) acc[v] = 0.0;
    for (int base = 0; base < n_chunks; base += kNormThreads) {
      uint4 hv8[kNormThreads / 32];
#pragma unroll
      for (int v = 0; v < kNormThreads / 32; ++v) {
        const int c = base + 32 * v + lane;
        hv8[v] = c < n_chunks ? __ldg(src4 + c) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int v = 0; v < kNormThreads / 32; ++v) {
        const int c = base + 32 * v + lane;
        if (c < n_chunks) {
          const uint4 hv = hv8[v];
          const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t ul = (w[j] & 0x7fffu) << 13, uh = (w[j] & 0x7fff0000u) >> 3;
            umin = min(umin, min(ul, uh));
            const double lo = __hiloint2double((int)(ul + 0x38000000u), 0);
            const double hi = __hiloint2double((int)(uh + 0x38000000u), 0);
            acc[v] += lo * lo;
            acc[v] += hi * hi;
          }
        }
      }
    }
    double tot = 0.0;
#pragma unroll
    for (int v = 0; v < kNormThreads / 32; ++v) {
#pragma unroll
      for (int m = 16; m; m >>= 1) acc[v] += __shfl_xor_sync(0xffffffffu, acc[v], m);
      tot += acc[v];
    }
    int redo = umin < 0x00100000u;                 // an element with exponent field 0
#pragma unroll
    for (int m = 16; m; m >>= 1) redo |= __shfl_xor_sync(0xffffffffu, redo, m);
    if (!redo && tot < 0x1p256) {                  // no Inf/NaN pattern either
      const double inv = 1.0 / sqrt(tot);
      // eight chunks per lane at a time, their loads issued together (the row comes from L2)
      for (int base = 0; base < n_chunks; base += kNormThreads) {
        uint4 hv[kNormThreads / 32];
#pragma unroll
        for (int v = 0; v < kNormThreads / 32; ++v) {
          const int c = base + 32 * v + lane;
          hv[v] = c < n_chunks ? __ldg(src4 + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int v = 0; v < kNormThreads / 32; ++v) {
          const int c = base + 32 * v + lane;
          if (c >= n_chunks) continue;
          const uint32_t w[4] = {hv[v].x, hv[v].y, hv[v].z, hv[v].w};
          uint32_t o[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t hl = ((w[j] & 0x8000u) << 16) | (((w[j] & 0x7fffu) << 13) + 0x38000000u);
            const uint32_t hh = (w[j] & 0x80000000u) | (((w[j] & 0x7fff0000u) >> 3) + 0x38000000u);
            const float lo = __double2float_rn(__hiloint2double((int)hl, 0) * inv);
            const float hi = __double2float_rn(__hiloint2double((int)hh, 0) * inv);
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[j]) : "f"(hi), "f"(lo));
          }
          dst4[c] = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
      return kRowOk;
    }
  }
  // every other row: conversions for all elements, Inf/NaN found from the bits
  double acc[kNormThreads / 32];
  int bad = 0;
#pragma unroll
  for (int v = 0; v < kNormThreads / 32; ++v) acc[v] = 0.0;
  for (int base = 0; base < n_chunks; base += kNormThreads) {
#pragma unroll
    for (int v = 0; v < kNormThreads / 32; ++v) {
      const int c = base + 32 * v + lane;
      if (c < n_chunks) {
        const uint4 hv = __ldg(src4 + c);
        const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float lo = bf16_lo(w[j]), hi = bf16_hi(w[j]);
          bad |= ((w[j] & 0x7f80u) == 0x7f80u) | ((w[j] & 0x7f800000u) == 0x7f800000u);
          acc[v] += (double)lo * (double)lo;
          acc[v] += (double)hi * (double)hi;
        }
      }
    }
  }
  double tot = 0.0;
#pragma unroll
  for (int v = 0; v < kNormThreads / 32; ++v) {
#pragma unroll
    for (int m = 16; m; m >>= 1) acc[v] += __shfl_xor_sync(0xffffffffu, acc[v], m);
    tot += acc[v];
  }
#pragma unroll
  for (int m = 16; m; m >>= 1) bad |= __shfl_xor_sync(0xffffffffu, bad, m);
  const double nrm = sqrt(tot);
  const bool ok = !bad && nrm > 0.0 && isfinite(nrm);
  const double inv = ok ? 1.0 / nrm : 0.0;
  for (int c = lane; c < n_chunks; c += 32) {
    const uint4 hv = __ldg(src4 + c);
    const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (inv == 0.0) { o[j] = 0; continue; }
      const float lo = __double2float_rn((double)bf16_lo(w[j]) * inv);
      const float hi = __double2float_rn((double)bf16_hi(w[j]) * inv);
      o[j] = f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
    }
    dst4[c] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  return ok ? kRowOk : ((bad || !isfinite(nrm)) ? kRowNonFinite : kRowZero);
}

// NT = number of 8-query tiles a pass scores (1: up to 8 queries, 2: up to 16).  One CTA of
// four quads (16 warps) per SM: it holds the normalised queries once (two CTAs of two quads,
// each with its own copy, were measured 3-15 % slower at every width, and rows wider than 6144
// elements leave no room for two copies), leaves half as many lists to the final merge, and
// its row share splits evenly over the quads.
// kFp8: the pool holds E4M3 codes + one fp32 scale per row (16 elements per 16-byte load, four
// f16 MMAs per pair of loads; score = scale * sum, as in the CUDA-core scan of such pools).
template <int E, int NT, bool kFp8>
__global__ void __launch_bounds__(kMmaThreads, 1)
scan_mma_kernel(PoolView pv, const uint8_t* __restrict__ codes, const float* __restrict__ scales,
                const uint16_t* __restrict__ q_raw, int nq, int k,
                const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                int32_t* __restrict__ q_valid, DeviceStats* stats, FusedAppend fa) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int KK = 32 * E;
  constexpr int QP = kMmaQ * NT;             // queries per pass
  constexpr int kQuads = kMmaThreads / 128;  // quads of four warps per CTA
  constexpr int kMmaDepth = NT == 1 ? kMmaDepth1 : kMmaDepth2;
  pdl_enter();   // the rows appended before this query, and the query states themselves
  const int d = pv.d, n_chunks = d >> 3;
  const int k_units = kFp8 ? d >> 4 : d >> 3;                            // 16-byte units of a key row
  const int q_stride = n_chunks + kMmaPadBytes / 16;                     // in 16-byte units
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                        // [QP][q_stride]
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)QP * q_stride * 16);   // [quads][QP][KK]
  // partial scores of a group: [buffer][quad][quarter][tile][lane]
  float4* s_part = reinterpret_cast<float4*>(smem_raw + (size_t)QP * q_stride * 16 +
                                             (size_t)kQuads * QP * KK * sizeof(u64));
  __shared__ uint64_t s_ex[QP];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  // contiguous, balanced share of the rows for this CTA
  const int64_t n = pv.n_rows;
  const int r_lo = (int)((n * blockIdx.x) / gridDim.x);
  const int r_hi = (int)((n * (blockIdx.x + 1)) / gridDim.x);
  const uint4* keys4 = kFp8 ? reinterpret_cast<const uint4*>(codes)
                            : reinterpret_cast<const uint4*>(pv.keys);

  // the step's append (Section 4 "(i) Store", Eq. 1): in the 8-query form warps 8 to 15 have
  // no query to prepare, so each of them in the first CTAs normalises one row meanwhile
  // (row 8 b + w - 8 in CTA b), with the numbers of the block routine, and counts it in
  if (!kFp8 && NT == 1 && warp >= 8 && (int)blockIdx.x * 8 + (warp - 8) < fa.n) {
    const int r = blockIdx.x * 8 + (warp - 8);
    const int64_t row = (int64_t)fa.row0 + r;
    const int code = normalize_row_warp(fa.states + (size_t)r * d, fa.keys + row * d, d, lane);
    if (lane == 0) {
      fa.tok[row] = fa.tokens[r];
      fa.trace_id[row] = fa.trace;
      if (code != kRowOk) atomicAdd(&stats->degenerate_rows, 1ull);  // stored as a zero key
      if (r == 0) {
        fa.trace_end[fa.trace] = fa.row0 + fa.n;
        if (fa.set_tag) { fa.trace_tag[fa.trace] = fa.tag; fa.trace_gbase[fa.trace] = fa.gbase; }
      }
    }
    __threadfence();                   // this lane's part of the row, before the count
    __syncwarp();
    if (lane == 0) {
      __threadfence();                 // cumulative: the whole warp's row, as seen through the barrier
      atomicAdd(fa.ready, 1ull);
    }
  }
  // 8-bit pools: the same eight warps quantise one row per CTA together (the block routine,
  // meeting at a named barrier of their own)
  if (kFp8 && NT == 1 && warp >= 8 && (int)blockIdx.x < fa.n) {
    const int r = blockIdx.x;
    const int64_t row = (int64_t)fa.row0 + r;
    const bool ok = quantize_row_e4m3<true, 256, 5>(fa.states + (size_t)r * d, d,
                                                    const_cast<uint8_t*>(codes) + row * d,
                                                    const_cast<float*>(scales) + row);
    if (threadIdx.x == 256) {
      fa.tok[row] = fa.tokens[r];
      fa.trace_id[row] = fa.trace;
      if (!ok) atomicAdd(&stats->degenerate_rows, 1ull);           // stored as a zero key
      if (r == 0) {
        fa.trace_end[fa.trace] = fa.row0 + fa.n;
        if (fa.set_tag) { fa.trace_tag[fa.trace] = fa.tag; fa.trace_gbase[fa.trace] = fa.gbase; }
      }
    }
    __threadfence();                   // this thread's part of the row, before the count
    asm volatile("bar.sync 5, 256;" ::: "memory");
    if (threadIdx.x == 256) {
      __threadfence();                 // cumulative: the eight warps' row, as seen through the barrier
      atomicAdd(fa.ready, 1ull);
    }
  }
  bool waited = fa.n == 0;             // this warp has seen the appended rows arrive
  // a group of rows that holds rows of this step's append: read through L2, after the wait
  auto fresh_at = [&](int rbx) { return fa.n > 0 && rbx + kMmaRows > fa.row0; };

  for (int q0 = 0; q0 < nq; q0 += QP) {
    __syncthreads();
    // query preparation, one warp per query: qs[w] = bf16(q / ||q||), exactly as a key is stored
    if (warp < QP) {
      uint16_t* dst = reinterpret_cast<uint16_t*>(qs + (size_t)warp * q_stride);
      if (q0 + warp < nq) {
        const int code = normalize_row_warp(q_raw + (size_t)(q0 + warp) * d, dst, d, lane);
        if (kFp8) {
          // the normalised bf16 query, as f16 scaled by 2^14 (exact but for elements below 2^-38)
          __syncwarp();
          uint32_t* w32 = reinterpret_cast<uint32_t*>(dst);
          for (int i = lane; i < d / 2; i += 32) {
            const uint32_t w = w32[i];
            const __half2 h = __floats2half2_rn(bf16_lo(w) * kFp8QueryScale, bf16_hi(w) * kFp8QueryScale);
            w32[i] = *reinterpret_cast<const uint32_t*>(&h);
          }
        }
        if (blockIdx.x == 0 && lane == 0) {
          q_valid[q0 + warp] = code == kRowNonFinite ? 0 : 1;   // NaN/Inf: no neighbours
          if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
        }
      } else {
        for (int c = lane; c < n_chunks; c += 32) qs[(size_t)warp * q_stride + c] = make_uint4(0, 0, 0, 0);
      }
      if (lane == 0)
        s_ex[warp] = (exclude_tag && q0 + warp < nq) ? exclude_tag[q0 + warp] : 0;
    }
    __syncthreads();

    // Four warps (a quad) share a group of 16 rows, every fourth 32-element block of the row
    // width each (so that the quad reads a row in contiguous kilobytes); the four partial
    // sums meet in shared memory and every warp adds them up.  A warp alone on a
    // group would leave a CTA's 200-odd rows of a paper-size pool as 14 units for 8 warps
    // (two rounds, the second three-quarters empty); as 7 units per quad the rounds are full.
    // The lists are shared out as well: warp kq of a quad keeps those of queries 2 kq and
    // 2 kq + 1 of every tile (the scores its lanes with t == kq hold), over all rows of the
    // quad, so a list sees four times the rows a per-warp list would and far fewer rows pass.
    const int quad = warp >> 2, kq = warp & 3;
    const int cq = k_units >> 2;                                    // 16-byte key units per quarter
    // query fragments: the 16 bytes (8 elements) that go with a 16-byte key unit, two of them
    // for a unit of 16 codes; tile i: + 8 i rows
    const uint4* qrow = qs + (size_t)g * q_stride + (kFp8 ? 2 : 1) * (kq * 4 + t);
    float4* part = s_part + quad * 4 * NT * 32;                     // [quarter][tile][lane]
    // descending lists of this warp's 2 NT queries; kth = the k-th entry (0 while not full)
    u64 top[2 * NT][E];
    u64 kth[2 * NT];
    const bool own = t == kq;                                       // this lane's scores are this warp's
#pragma unroll
    for (int l = 0; l < 2 * NT; ++l) {
      kth[l] = 0;
#pragma unroll
      for (int r = 0; r < E; ++r) top[l][r] = 0;
    }
    int buf = 0;

    // key pointers of this lane's two rows of the group starting at row rbx
    auto row_ptr = [&](int rbx, int second) {
      const int row = rbx + g + 8 * second;
      return keys4 + (size_t)(row < r_hi ? row : r_hi - 1) * k_units + kq * 4 + t;
    };
    // The key stream of a warp is one sequence of steps of kMmaDepth blocks of 32 elements
    // over all its groups: the loads of the next step (the first of the next group, at a
    // group's end) are issued before this step's MMAs, so that the loads in flight never
    // drain, neither while the tensor pipe works nor across a group's epilogue.
    int rb = r_lo + quad * kMmaRows;
    const uint4 *pa = keys4, *pb = keys4;
    uint4 ka[kMmaDepth], kb[kMmaDepth];
    bool cur_fresh = rb < r_hi && fresh_at(rb);
    if (rb < r_hi) {
      if (cur_fresh && !waited) {
        wait_fused_rows(fa, stats);
        waited = true;
      }
      pa = row_ptr(rb, 0);
      pb = row_ptr(rb, 1);
#pragma unroll
      for (int u = 0; u < kMmaDepth; ++u) {
        const bool in = 4 * u < cq;
        ka[u] = in ? ld_key16(pa + 4 * (4 * u), cur_fresh) : make_uint4(0, 0, 0, 0);
        kb[u] = in ? ld_key16(pb + 4 * (4 * u), cur_fresh) : make_uint4(0, 0, 0, 0);
      }
    }
    for (; rb < r_hi; rb += kQuads * kMmaRows) {
      const int row0 = rb + g, row1 = rb + g + 8;
      // 8-bit pools: the rows' scales (and the queries' 2^14 taken back), asked for before the
      // group's arithmetic so that the epilogue does not wait a round trip for them (a group
      // that holds rows appended by this launch has waited for them before its first load)
      float sc0 = 1.f, sc1 = 1.f;
      if (kFp8 && own) {
        // (a row appended by this launch: its scale was written a moment ago, read it through L2)
        sc0 = row0 < r_hi ? (cur_fresh ? __ldcg(&scales[row0]) : scales[row0]) * (1.f / kFp8QueryScale) : 0.f;
        sc1 = row1 < r_hi ? (cur_fresh ? __ldcg(&scales[row1]) : scales[row1]) * (1.f / kFp8QueryScale) : 0.f;
      }
      const bool has_next = rb + kQuads * kMmaRows < r_hi;
      const bool next_fresh = has_next && fresh_at(rb + kQuads * kMmaRows);
      // the next group's first step is fetched early unless it holds rows that this launch
      // appends and the wait for them is still ahead
      const bool pre_next = has_next && (!next_fresh || waited);
      const uint4* pna = has_next ? row_ptr(rb + kQuads * kMmaRows, 0) : pa;
      const uint4* pnb = has_next ? row_ptr(rb + kQuads * kMmaRows, 1) : pb;
      float c0[NT][4], c1[NT][4];
#pragma unroll
      for (int i = 0; i < NT; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) c0[i][e] = c1[i][e] = 0.f;
      // the steps of a group; kMixed = some of its loads (its own or the next group's first
      // step) go to rows appended by this launch and must not use the read-only path
      auto run_steps = [&](auto mixed) {
        constexpr bool kMixed = decltype(mixed)::value;
        for (int c = 0; c < cq; c += 4 * kMmaDepth) {
          uint4 na[kMmaDepth], nb[kMmaDepth];
          const int cn = c + 4 * kMmaDepth;
          const bool same = cn < cq;                       // next step: same group or the next one
          const uint4* sa = same ? pa + 4 * cn : pna;
          const uint4* sb = same ? pb + 4 * cn : pnb;
          const int left = same ? cq - cn : (pre_next ? cq : 0);
          const bool ld_fresh = kMixed && (same ? cur_fresh : next_fresh);
#pragma unroll
          for (int u = 0; u < kMmaDepth; ++u) {
            const bool in = 4 * u < left;
            if (kMixed) {
              na[u] = in ? ld_key16(sa + 4 * (4 * u), ld_fresh) : make_uint4(0, 0, 0, 0);
              nb[u] = in ? ld_key16(sb + 4 * (4 * u), ld_fresh) : make_uint4(0, 0, 0, 0);
            } else {
              na[u] = in ? ld_stream16(sa + 4 * (4 * u)) : make_uint4(0, 0, 0, 0);
              nb[u] = in ? ld_stream16(sb + 4 * (4 * u)) : make_uint4(0, 0, 0, 0);
            }
          }
#pragma unroll
          for (int u = 0; u < kMmaDepth; ++u) {
#pragma unroll
            for (int i = 0; i < NT; ++i) {
              if (kFp8) {
                const bool in = c + 4 * u < cq;
                const uint4* qp = qrow + (size_t)8 * i * q_stride + 8 * (c + 4 * u);
                const uint4 ql = in ? qp[0] : make_uint4(0, 0, 0, 0);
                const uint4 qh = in ? qp[1] : make_uint4(0, 0, 0, 0);
                mma_f16(c0[i], e4m3x2_to_f16x2(ka[u].x), e4m3x2_to_f16x2(kb[u].x),
                        e4m3x2_to_f16x2(ka[u].x >> 16), e4m3x2_to_f16x2(kb[u].x >> 16), ql.x, ql.y);
                mma_f16(c1[i], e4m3x2_to_f16x2(ka[u].y), e4m3x2_to_f16x2(kb[u].y),
                        e4m3x2_to_f16x2(ka[u].y >> 16), e4m3x2_to_f16x2(kb[u].y >> 16), ql.z, ql.w);
                mma_f16(c0[i], e4m3x2_to_f16x2(ka[u].z), e4m3x2_to_f16x2(kb[u].z),
                        e4m3x2_to_f16x2(ka[u].z >> 16), e4m3x2_to_f16x2(kb[u].z >> 16), qh.x, qh.y);
                mma_f16(c1[i], e4m3x2_to_f16x2(ka[u].w), e4m3x2_to_f16x2(kb[u].w),
                        e4m3x2_to_f16x2(ka[u].w >> 16), e4m3x2_to_f16x2(kb[u].w >> 16), qh.z, qh.w);
              } else {
                const uint4 qv = c + 4 * u < cq ? qrow[(size_t)8 * i * q_stride + 4 * (c + 4 * u)]
                                                : make_uint4(0, 0, 0, 0);
                mma_bf16(c0[i], ka[u].x, kb[u].x, ka[u].y, kb[u].y, qv.x, qv.y);
                mma_bf16(c1[i], ka[u].z, kb[u].z, ka[u].w, kb[u].w, qv.z, qv.w);
              }
            }
          }
#pragma unroll
          for (int u = 0; u < kMmaDepth; ++u) { ka[u] = na[u]; kb[u] = nb[u]; }
        }
      };
      if (cur_fresh || next_fresh) run_steps(BoolTrue{});
      else run_steps(BoolFalse{});
      pa = pna;
      pb = pnb;
      // partial scores of (row0, 2t), (row0, 2t+1), (row1, 2t), (row1, 2t+1) of every tile.
      // Two buffers, one barrier per group: a warp reads a group's partials before it starts
      // the next group, so when it arrives here for group i it is done with group i - 1, and
      // the barrier of group i - 1 has shown that everyone was done with group i - 2
      float4* pbuf = part + (buf ? kQuads * 4 * NT * 32 : 0);
      buf ^= 1;
#pragma unroll
      for (int i = 0; i < NT; ++i)
        pbuf[(kq * NT + i) * 32 + lane] = make_float4(c0[i][0] + c1[i][0], c0[i][1] + c1[i][1],
                                                      c0[i][2] + c1[i][2], c0[i][3] + c1[i][3]);
      quad_bar(1 + quad);                    // this group's partials are in
      uint64_t tag0 = 0, tag1 = 0;
      if (exclude_tag && own) {
        // rows appended by this launch: their trace id and tag were written by another CTA a
        // moment ago, so those are read through L2
        if (row0 < r_hi)
          tag0 = cur_fresh ? __ldcg(&pv.trace_tag[__ldcg(&pv.trace_id[row0])]) : pv.trace_tag[pv.trace_id[row0]];
        if (row1 < r_hi)
          tag1 = cur_fresh ? __ldcg(&pv.trace_tag[__ldcg(&pv.trace_id[row1])]) : pv.trace_tag[pv.trace_id[row1]];
      }
      u64 key[2 * NT][2];                    // [list][row0 / row1]
      bool any = false;
#pragma unroll
      for (int i = 0; i < NT; ++i) {
        const float4 p0 = pbuf[(0 * NT + i) * 32 + lane], p1 = pbuf[(1 * NT + i) * 32 + lane],
                     p2 = pbuf[(2 * NT + i) * 32 + lane], p3 = pbuf[(3 * NT + i) * 32 + lane];
        float sx = ((p0.x + p1.x) + p2.x) + p3.x, sy = ((p0.y + p1.y) + p2.y) + p3.y;
        float sz = ((p0.z + p1.z) + p2.z) + p3.z, sw = ((p0.w + p1.w) + p2.w) + p3.w;
        if (kFp8) { sx *= sc0; sy *= sc0; sz *= sc1; sw *= sc1; }
        const int la = 2 * i, lb = 2 * i + 1;
        const int qa = 8 * i + 2 * kq;                     // queries of lists la, lb within the pass
        const bool live_a = own && q0 + qa < nq, live_b = own && q0 + qa + 1 < nq;
        // exclusion tags are read where they are used: they are rare, registers are not
        const uint64_t ex_a = exclude_tag ? s_ex[qa] : 0, ex_b = exclude_tag ? s_ex[qa + 1] : 0;
        key[la][0] = (row0 < r_hi && live_a && !(ex_a != 0 && tag0 == ex_a)) ? pack_candidate(sx, (uint32_t)row0) : 0;
        key[lb][0] = (row0 < r_hi && live_b && !(ex_b != 0 && tag0 == ex_b)) ? pack_candidate(sy, (uint32_t)row0) : 0;
        key[la][1] = (row1 < r_hi && live_a && !(ex_a != 0 && tag1 == ex_a)) ? pack_candidate(sz, (uint32_t)row1) : 0;
        key[lb][1] = (row1 < r_hi && live_b && !(ex_b != 0 && tag1 == ex_b)) ? pack_candidate(sw, (uint32_t)row1) : 0;
        any |= (key[la][0] > kth[la]) | (key[la][1] > kth[la]) | (key[lb][0] > kth[lb]) | (key[lb][1] > kth[lb]);
      }
      if (__any_sync(0xffffffffu, any)) {
#pragma unroll
        for (int l = 0; l < 2 * NT; ++l) {
          const unsigned b0 = __ballot_sync(0xffffffffu, key[l][0] > kth[l]);
          const unsigned b1 = __ballot_sync(0xffffffffu, key[l][1] > kth[l]);
          if (__popc(b0) + __popc(b1) >= kMmaBatchInsert) {
            // many rows pass (a list's first groups): the group's 16 scores of this query
            // are sorted as one vector and merged in, which costs about four insertions
            const int src = (lane & 7) * 4 + kq;
            const uint32_t l0 = __shfl_sync(0xffffffffu, (uint32_t)key[l][0], src);
            const uint32_t h0 = __shfl_sync(0xffffffffu, (uint32_t)(key[l][0] >> 32), src);
            const uint32_t l1 = __shfl_sync(0xffffffffu, (uint32_t)key[l][1], src);
            const uint32_t h1 = __shfl_sync(0xffffffffu, (uint32_t)(key[l][1] >> 32), src);
            u64 v[1];
            v[0] = lane < 8 ? (((u64)h0 << 32) | l0) : lane < 16 ? (((u64)h1 << 32) | l1) : 0;
            v[0] = v[0] > kth[l] ? v[0] : 0;
            warp_sort_desc<1>(v, lane);
            u64 add[E];
            add[0] = v[0];
#pragma unroll
            for (int r = 1; r < E; ++r) add[r] = 0;
            warp_merge_desc<E>(top[l], add, lane);
            kth[l] = warp_list_get<E>(top[l], k - 1);
            continue;
          }
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const u64 mine = key[l][half];
            unsigned b = half ? b1 : b0;
            while (b) {
              const int src = __ffs(b) - 1;
              b &= b - 1;
              const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)mine, src);
              const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)(mine >> 32), src);
              const u64 cand = ((u64)hi << 32) | lo;
              if (cand > kth[l]) {
                warp_sorted_insert<E>(top[l], cand, lane);
                kth[l] = warp_list_get<E>(top[l], k - 1);
              }
            }
          }
        }
      }
      if (has_next && !pre_next) {
        // the next group holds rows of this step's append: wait (bounded) until all of them
        // are in, then fetch its first step
        wait_fused_rows(fa, stats);
        waited = true;
#pragma unroll
        for (int u = 0; u < kMmaDepth; ++u) {
          const bool in = 4 * u < cq;
          ka[u] = in ? ld_key16(pa + 4 * (4 * u), true) : make_uint4(0, 0, 0, 0);
          kb[u] = in ? ld_key16(pb + 4 * (4 * u), true) : make_uint4(0, 0, 0, 0);
        }
      }
      cur_fresh = next_fresh;
    }

    // warp w merges the quads' lists of query w and publishes the CTA's KK best
    __syncthreads();
#pragma unroll
    for (int l = 0; l < 2 * NT; ++l) {
      const int qi = 8 * (l >> 1) + 2 * kq + (l & 1);
#pragma unroll
      for (int r = 0; r < E; ++r)
        scratch[((size_t)quad * QP + qi) * KK + r * 32 + lane] = top[l][r];
    }
    __syncthreads();
    if (warp < QP && q0 + warp < nq) {
      u64 a[E];
#pragma unroll
      for (int r = 0; r < E; ++r) a[r] = scratch[((size_t)0 * QP + warp) * KK + r * 32 + lane];
      for (int qd = 1; qd < kQuads; ++qd) {
        u64 b[E];
#pragma unroll
        for (int r = 0; r < E; ++r) b[r] = scratch[((size_t)qd * QP + warp) * KK + r * 32 + lane];
        warp_merge_desc<E>(a, b, lane);
      }
      u64* dst = partial + ((size_t)blockIdx.x * nq + (q0 + warp)) * KK;
#pragma unroll
      for (int r = 0; r < E; ++r) dst[r * 32 + lane] = a[r];
    }
  }
}

size_t scan_mma_smem(int32_t d, int32_t kk, int32_t nt) {
  const size_t qp = (size_t)kMmaQ * nt, quads = kMmaThreads / 128;
  return qp * ((size_t)d * 2 + kMmaPadBytes) + quads * qp * kk * sizeof(u64) +
         2 * quads * 4 * nt * 32 * sizeof(float4);
}

// 8-query tiles per pass (1 or 2) for a call of nq queries, or 0 if the kernel cannot take
// the pool's width (a quad's warps take whole blocks of 32 elements, 64 codes for 8-bit
// keys) or the list length
int scan_mma_tiles(int32_t d, int32_t kk, int32_t nq, size_t smem_limit, bool fp8) {
  if (d % (fp8 ? 256 : 128) != 0 || kk > 64) return 0;
  if (nq > kMmaQ && scan_mma_smem(d, kk, 2) <= smem_limit) return 2;
  return scan_mma_smem(d, kk, 1) <= smem_limit ? 1 : 0;
}

bool scan_mma_supports(int32_t d, int32_t kk, size_t smem_limit, bool fp8) {
  return scan_mma_tiles(d, kk, 1, smem_limit, fp8) != 0;
}

// CTAs the scan launches: at least 64 rows each, at most one per SM
int32_t scan_mma_grid(int64_t n_rows, int32_t num_sms, int32_t max_lists) {
  const int64_t want = (n_rows + 63) / 64;
  const int32_t grid = (int32_t)(want < 1 ? 1 : (want > num_sms ? num_sms : want));
  return grid > max_lists ? max_lists : grid;
}

template <int E, int NT, bool kFp8>
static cudaError_t launch_mma_one(const PoolView& pv, const uint8_t* codes, const float* scales,
                                  const uint16_t* q_raw, int nq, int k, const uint64_t* ex,
                                  u64* partial, int32_t* q_valid, DeviceStats* stats, int grid,
                                  const FusedAppend& fa, cudaStream_t st) {
  const size_t smem = scan_mma_smem(pv.d, 32 * E, NT);
  return launch_pdl(scan_mma_kernel<E, NT, kFp8>, dim3(grid), dim3(kMmaThreads), smem, st, pv, codes,
                    scales, q_raw, nq, k, ex, partial, q_valid, stats, fa);
}

cudaError_t launch_scan_mma(const PoolView& pv, const uint8_t* codes, const float* scales,
                            const uint16_t* q_raw, int32_t nq, int32_t k, int32_t kk,
                            const uint64_t* exclude_tag, u64* partial, int32_t* q_valid,
                            DeviceStats* stats, int32_t max_lists, int32_t num_sms,
                            size_t smem_limit, int32_t* n_lists, const FusedAppend* fused,
                            cudaStream_t st) {
  const bool fp8 = codes != nullptr;
  const int nt = scan_mma_tiles(pv.d, kk, nq, smem_limit, fp8);
  if (nt == 0) return cudaErrorInvalidValue;
  const int grid = scan_mma_grid(pv.n_rows, num_sms, max_lists);
  *n_lists = grid;
  FusedAppend fa = {};
  if (fused) {
    // every appending warp must exist (eight per CTA), and all CTAs be resident together
    // (they are: at most one per SM is launched), because scanning warps wait for the
    // appending ones; the 8-query form only (8-bit keys: one row per CTA)
    if (nt != 1 || fused->n > (fp8 ? 1 : 8) * grid || fused->n > kFuseMaxRows) return cudaErrorInvalidValue;
    fa = *fused;
  }
#define OILBIRD_MMA_CASE(E_, NT_, F_)                                                          \
  if (kk == 32 * E_ && nt == NT_ && fp8 == F_)                                                 \
    return launch_mma_one<E_, NT_, F_>(pv, codes, scales, q_raw, nq, k, exclude_tag, partial,  \
                                       q_valid, stats, grid, fa, st);
  OILBIRD_MMA_CASE(1, 1, false)
  OILBIRD_MMA_CASE(2, 1, false)
  OILBIRD_MMA_CASE(1, 2, false)
  OILBIRD_MMA_CASE(2, 2, false)
  OILBIRD_MMA_CASE(1, 1, true)
  OILBIRD_MMA_CASE(2, 1, true)
  OILBIRD_MMA_CASE(1, 2, true)
  OILBIRD_MMA_CASE(2, 2, true)
#undef OILBIRD_MMA_CASE
  return cudaErrorInvalidValue;
}

cudaError_t preload_scan_mma_kernels() {
  cudaError_t e;
  if ((e = preload_kernel(scan_mma_kernel<1, 1, false>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_mma_kernel<2, 1, false>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_mma_kernel<1, 2, false>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_mma_kernel<2, 2, false>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_mma_kernel<1, 1, true>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_mma_kernel<2, 1, true>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_mma_kernel<1, 2, true>, true)) != cudaSuccess) return e;
  return preload_kernel(scan_mma_kernel<2, 2, true>, true);
}

}  // namespace oilbird
