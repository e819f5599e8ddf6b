// L2 normalisation of one bf16 row, shared by the append kernel (keys, Eq. 1: states are
// stored normalised in 16-bit precision) and by query preparation (the cosine of
// Algorithm 1's scoring line then is a plain dot product of two stored-format vectors).
#pragma once
#include "common.cuh"

namespace oilbird {

constexpr int kNormThreads = 256;

enum { kRowOk = 0, kRowZero = 1, kRowNonFinite = 2 };

// Load the first kHeld chunks per thread of a row into registers (zero past the row's end).
template <int kHeld>
__device__ __forceinline__ void load_row_chunks(const uint16_t* __restrict__ src, int d,
                                                uint4 (&held)[kHeld]) {
  const int n_chunks = d >> 3;
  const uint4* src4 = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int i = 0; i < kHeld; ++i) {
    const int c = threadIdx.x + i * kNormThreads;
    held[i] = c < n_chunks ? __ldg(src4 + c) : make_uint4(0, 0, 0, 0);
  }
}

// The arithmetic of normalize_row on a row whose first kHeld chunks per thread the caller
// has loaded already (load_row_chunks), so that a kernel looping over rows can issue the
// next row's loads before it reduces this one.
template <bool kHold, int kHeld, bool kFast = false>
__device__ __forceinline__ int normalize_row_regs(const uint4 (&held)[kHeld],
                                                  const uint16_t* __restrict__ src,
                                                  uint16_t* __restrict__ dst, int d) {
  __shared__ double s_part[kNormThreads / 32];
  __shared__ int s_bad[kNormThreads / 32];
  __shared__ double s_inv;
  __shared__ int s_code;
  const int n_chunks = d >> 3;
  const uint4* src4 = reinterpret_cast<const uint4*>(src);
  // at most 8 chunks of 8 elements per thread (d <= 16384); the first kHeld of them stay
  // in registers so that a row of up to kHeld * 2048 elements is read from memory once
  constexpr int kMaxChunks = 16384 / 8 / kNormThreads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint4* dst4 = reinterpret_cast<uint4*>(dst);

  // Fast path, for rows whose elements are all normal finite numbers (every row of real
  // hidden states).  The float->double conversion instruction runs at a quarter of the
  // arithmetic rate, and three of them per element (two up, one down) bounded the kernel
  // below the memory system's speed.  A normal bf16 value's double is built from its bits
  // instead: exponent field e + 896, the 7 fraction bits on top of the double's 52, low word
  // zero.  That is the value the conversion gives, so sums, scale and products are the same
  // numbers in the same order as on the exact path below.  The smallest biased exponent seen
  // tells whether a zero or subnormal was among the elements, and a sum of 2^256 or more
  // that an Inf/NaN pattern may have been (read as 2^128 and up); such rows, zero rows among
  // them, are redone on the exact path.  kFast is set by the kernels that normalise rows in
  // bulk; where one or a few rows sit in front of other work (query preparation, the rows a
  // scan appends) the kernel is bound by latency and the extra code only costs.
  if (kFast) {
    double fs = 0.0;
    uint32_t umin = 0xffffffffu;
#pragma unroll
    for (int i = 0; i < kMaxChunks; ++i) {
      const int c0 = threadIdx.x + i * kNormThreads;
      if (c0 >= n_chunks) break;
      const uint4 hv = (kHold && i < kHeld) ? held[i] : __ldg(src4 + c0);
      const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t ul = (w[j] & 0x7fffu) << 13, uh = (w[j] & 0x7fff0000u) >> 3;
        umin = min(umin, min(ul, uh));
        const double lo = __hiloint2double((int)(ul + 0x38000000u), 0);
        const double hi = __hiloint2double((int)(uh + 0x38000000u), 0);
        fs += lo * lo;
        fs += hi * hi;
      }
    }
    int redo = umin < 0x00100000u;      // an element with exponent field 0
#pragma unroll
    for (int m = 16; m; m >>= 1) {
      fs += __shfl_xor_sync(0xffffffffu, fs, m);
      redo |= __shfl_xor_sync(0xffffffffu, redo, m);
    }
    if (lane == 0) { s_part[warp] = fs; s_bad[warp] = redo; }
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = 0.0;
      int b = 0;
      for (int w = 0; w < kNormThreads / 32; ++w) { tot += s_part[w]; b |= s_bad[w]; }
      b |= !(tot < 0x1p256);
      s_inv = b ? 0.0 : 1.0 / sqrt(tot);
      s_code = b ? -1 : kRowOk;
    }
    __syncthreads();
    if (s_code == kRowOk) {
      const double inv = s_inv;
#pragma unroll
      for (int i = 0; i < kMaxChunks; ++i) {
        const int c = threadIdx.x + i * kNormThreads;
        if (c >= n_chunks) break;
        const uint4 hv = (kHold && i < kHeld) ? held[i] : __ldg(src4 + c);
        const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t hl = ((w[j] & 0x8000u) << 16) | (((w[j] & 0x7fffu) << 13) + 0x38000000u);
          const uint32_t hh = (w[j] & 0x80000000u) | (((w[j] & 0x7fff0000u) >> 3) + 0x38000000u);
          const float lo = __double2float_rn(__hiloint2double((int)hl, 0) * inv);
          const float hi = __double2float_rn(__hiloint2double((int)hh, 0) * inv);
          // both halves rounded to nearest even and packed by one instruction
          asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[j]) : "f"(hi), "f"(lo));
        }
        dst4[c] = make_uint4(o[0], o[1], o[2], o[3]);
      }
      __syncthreads();   // the shared scratch may be reused by the next call
      return kRowOk;
    }
  }

  // Exact path for every other row: conversions for all elements, Inf/NaN found from the bits.
  double ss = 0.0;
  int bad = 0;
#pragma unroll
  for (int i = 0; i < kMaxChunks; ++i) {
    const int c0 = threadIdx.x + i * kNormThreads;
    if (c0 >= n_chunks) break;
    const uint4 hv = (kHold && i < kHeld) ? held[i] : __ldg(src4 + c0);
    const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float lo = bf16_lo(w[j]), hi = bf16_hi(w[j]);
      bad |= ((w[j] & 0x7f80u) == 0x7f80u) | ((w[j] & 0x7f800000u) == 0x7f800000u);
      ss += (double)lo * (double)lo;
      ss += (double)hi * (double)hi;
    }
  }
#pragma unroll
  for (int m = 16; m; m >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, m);
    bad |= __shfl_xor_sync(0xffffffffu, bad, m);
  }
  if (lane == 0) { s_part[warp] = ss; s_bad[warp] = bad; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    int b = 0;
    for (int w = 0; w < kNormThreads / 32; ++w) { tot += s_part[w]; b |= s_bad[w]; }
    double nrm = sqrt(tot);
    bool ok = !b && nrm > 0.0 && isfinite(nrm);
    s_inv = ok ? 1.0 / nrm : 0.0;
    s_code = ok ? kRowOk : ((b || !isfinite(nrm)) ? kRowNonFinite : kRowZero);
  }
  __syncthreads();
  const double inv = s_inv;
#pragma unroll
  for (int i = 0; i < kMaxChunks; ++i) {
    const int c = threadIdx.x + i * kNormThreads;
    if (c >= n_chunks) break;
    const uint4 hv = (kHold && i < kHeld) ? held[i] : __ldg(src4 + c);
    const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (inv == 0.0) { o[j] = 0; continue; }
      float lo = __double2float_rn((double)bf16_lo(w[j]) * inv);
      float hi = __double2float_rn((double)bf16_hi(w[j]) * inv);
      o[j] = f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
    }
    dst4[c] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  const int code = s_code;
  __syncthreads();   // the shared scratch may be reused by the next call
  return code;
}

// Two rows at once, fast path only (see normalize_row_regs): every chunk of both rows is in
// registers (d <= kHeld * 2048).  The per-row block reduction, its barriers and the square
// root and division that one thread does per row are the fixed cost of a row; two rows share
// the barriers, and threads 0 and 32 take one row's scale each.  Each row's numbers are
// accumulated in the order of the single-row routine, so the results are the same.  code_a /
// code_b come back as kRowOk, or -1 for a row that must be redone on the exact path (nothing
// has been written for it).
template <int kHeld>
__device__ __forceinline__ void normalize_two_rows_fast(const uint4 (&ha)[kHeld],
                                                        const uint4 (&hb)[kHeld],
                                                        uint16_t* __restrict__ dst_a,
                                                        uint16_t* __restrict__ dst_b, int d,
                                                        int& code_a, int& code_b) {
  __shared__ double s_part2[2][kNormThreads / 32];
  __shared__ int s_bad2[2][kNormThreads / 32];
  __shared__ double s_inv2[2];
  __shared__ int s_code2[2];
  const int n_chunks = d >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  double fs[2] = {0.0, 0.0};
  uint32_t umin[2] = {0xffffffffu, 0xffffffffu};
#pragma unroll
  for (int r = 0; r < 2; ++r) {
#pragma unroll
    for (int i = 0; i < kHeld; ++i) {
      if (threadIdx.x + i * kNormThreads >= n_chunks) break;
      const uint4 hv = r ? hb[i] : ha[i];
      const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t ul = (w[j] & 0x7fffu) << 13, uh = (w[j] & 0x7fff0000u) >> 3;
        umin[r] = min(umin[r], min(ul, uh));
        const double lo = __hiloint2double((int)(ul + 0x38000000u), 0);
        const double hi = __hiloint2double((int)(uh + 0x38000000u), 0);
        fs[r] += lo * lo;
        fs[r] += hi * hi;
      }
    }
  }
  int redo[2] = {umin[0] < 0x00100000u, umin[1] < 0x00100000u};
#pragma unroll
  for (int m = 16; m; m >>= 1) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      fs[r] += __shfl_xor_sync(0xffffffffu, fs[r], m);
      redo[r] |= __shfl_xor_sync(0xffffffffu, redo[r], m);
    }
  }
  if (lane == 0) {
    s_part2[0][warp] = fs[0]; s_bad2[0][warp] = redo[0];
    s_part2[1][warp] = fs[1]; s_bad2[1][warp] = redo[1];
  }
  __syncthreads();
  if (lane == 0 && warp < 2) {
    double tot = 0.0;
    int b = 0;
    for (int w = 0; w < kNormThreads / 32; ++w) { tot += s_part2[warp][w]; b |= s_bad2[warp][w]; }
    b |= !(tot < 0x1p256);
    s_inv2[warp] = b ? 0.0 : 1.0 / sqrt(tot);
    s_code2[warp] = b ? -1 : kRowOk;
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (s_code2[r] != kRowOk) continue;
    const double inv = s_inv2[r];
    uint4* dst4 = reinterpret_cast<uint4*>(r ? dst_b : dst_a);
#pragma unroll
    for (int i = 0; i < kHeld; ++i) {
      const int c = threadIdx.x + i * kNormThreads;
      if (c >= n_chunks) break;
      const uint4 hv = r ? hb[i] : ha[i];
      const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
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
  code_a = s_code2[0];
  code_b = s_code2[1];
  __syncthreads();   // the shared scratch is reused by the next pair
}

// Normalise one row of d bf16 values (d % 8 == 0) from src to dst (global or shared).
// All kNormThreads threads of the block take part.  The squared norm is accumulated in
// double precision (products of bf16 values are exact there), the scale 1/sqrt is IEEE
// double, each element is rounded once to float and once to bf16 (nearest even).
// Returns kRowOk, or kRowZero / kRowNonFinite, in which case dst is all zero.
// kHold: keep the row's first kHeld chunks per thread in registers between the two passes
// (one read of the row up to d = kHeld * 2048), or read it twice (for kernels that are short
// of registers).
template <bool kHold = true, int kHeld = 4, bool kFast = false>
__device__ __forceinline__ int normalize_row(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst,
                              int d) {
  uint4 held[kHeld];
  if (kHold) load_row_chunks<kHeld>(src, d, held);
  return normalize_row_regs<kHold, kHeld, kFast>(held, src, dst, d);
}

}  // namespace oilbird
