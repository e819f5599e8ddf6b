// 8-bit keys for a bounded store: append and CUDA-core scan for pools whose keys are
// FP8 E4M3 codes with one fp32 scale per row.
//
// The paper's Limitations section leaves "keeping the store bounded ... by eviction, an
// index, or quantization" as future work and fixes no format; the one implemented here:
//   v_j   = x_j / ||x||                       (double, as for 16-bit keys)
//   scale = fp32( max_j |v_j| / 448 )         (448 = largest finite E4M3 magnitude)
//   c_j   = e4m3_rne( v_j / scale )           (ties to the even code, saturating)
// and a score is fp32( scale * sum_j qn_j * value(c_j) ) with the query normalised and
// rounded to bf16 exactly as for 16-bit pools.  A row costs d + 4 bytes instead of 2d, so
// the scan, which is bound by the key stream, moves half the bytes.
//
// Everything after the scan (merge, firing rule, depth, gather) is format-independent and
// shared with the 16-bit path.  The tcgen05 scan is not offered for 8-bit pools (its query
// operand would have to be quantised to 8 bits too); batches of three queries and more go
// to the warp-level tensor scan (scan_mma.cu, codes as f16) where the width allows, else
// they run here two queries per pass.  As in the 16-bit scan, the rows of a serving step can be appended
// by the scan's first CTAs themselves (see FusedAppend).
#include <cuda_fp16.h>

#include "common.cuh"
#include "internal.h"
#include "normalize.cuh"

namespace oilbird {

// ---------------------------------------------------------------- E4M3 encode ---
// Nearest E4M3 code of t (double), ties to the even code, |t| >= 448 saturates to 448;
// the sign bit is kept even when the magnitude rounds to zero.
__device__ __forceinline__ uint32_t e4m3_encode(double t) {
  const uint32_t sign = (__double_as_longlong(t) < 0) ? 0x80u : 0u;
  const double a = fabs(t);
  if (!(a == a)) return 0;
  if (a >= 448.0) return sign | 0x7eu;
  if (a < 0.015625) {                                   // below 2^-6: spacing 2^-9
    const int n = (int)rint(a * 512.0);                 // 0..8; 8 is the smallest normal
    return sign | (uint32_t)n;
  }
  int e = ilogb(a);                                     // -6 .. 8
  int n = (int)rint(scalbn(a, 3 - e));                  // 8 .. 16, exact scaling
  if (n == 16) { n = 8; e += 1; }
  return sign | (uint32_t)(((e + 7) << 3) | (n - 8));
}

// The exact code of one element, out of line: the bulk quantiser reaches it for a few
// elements in a hundred thousand, and sixteen inlined copies per loop body would not fit the
// instruction cache.
__device__ __noinline__ uint32_t e4m3_encode_element(float x, double inv, double sc) {
  return e4m3_encode(((double)x * inv) / sc);
}

// --------------------------------------------------------------------- append ---
// Quantise one raw bf16 row (d a multiple of 16) into codes + scale.  All kNormThreads
// threads of the block take part; two passes over the row (it is re-read from L2):
// squared norm and peak, then the codes.  Returns true if the row was usable.
//
// kFast (the bulk append): rows whose elements are all normal finite numbers avoid the
// float<->double conversions, the double division and the general encoder, which together
// held the kernel at a sixth of the memory system's speed.
//  - the doubles are built from the bf16 bits (exponent field e + 896, fraction on top), the
//    peak is the largest magnitude pattern; sums, norm and scale are the same numbers in the
//    same order as on the exact path;
//  - per element t' = |x| * g with g = (1/||x||) / scale stands in for t = (|x| / ||x||) / scale.
//    The two differ by at most four units in the last place of a double, so they round to the
//    same code unless a rounding boundary of the code grid lies within that distance of t'.
//    Boundaries are numbers with five significant bits, so t' is near one when bits 16..0 of
//    its high word read 0xffff or 0x10000 and the low word is within 256 of wrapping.  (The
//    high-word pattern alone is common, 5 elements in a thousand: x and the peak are 8-bit
//    significands and the scale is their ratio rounded to float, which puts many t' within
//    2^-24 of a boundary; the low word separates those from the true near-ties.)  Near-ties
//    go through the exact encoder, out of line.
//  - for all others the code comes from the hardware: t' is handed over as a float that holds
//    its exponent, the 20 fraction bits of the double's high word and one sticky bit for the
//    rest, and cvt.rn.satfinite.e4m3x2.f32 rounds two of them to nearest even, subnormal
//    codes and the cap at 448 included.  (The sticky bit keeps the side of the boundary; a
//    plain double -> float conversion would round many of the common 2^-24 cases onto the
//    boundary itself.)  The four sign bits of a word of codes are picked from the inputs.
// A row with a zero, subnormal, Inf or NaN anywhere, or with an element more than 2^40 below
// its peak, is redone on the exact path.
template <bool kFast = false>
__device__ __forceinline__ bool quantize_row_e4m3(const uint16_t* __restrict__ src, int d,
                                                  uint8_t* __restrict__ dst, float* scale_out) {
  __shared__ double s_ss[kNormThreads / 32];
  __shared__ float s_mx[kNormThreads / 32];
  __shared__ int s_bad[kNormThreads / 32];
  __shared__ uint32_t s_lo[kNormThreads / 32];
  __shared__ double s_inv;
  __shared__ double s_g;
  __shared__ float s_scale;
  __shared__ int s_ok;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n16 = d >> 4;
  const uint4* src4 = reinterpret_cast<const uint4*>(src);
  uint4* dst4 = reinterpret_cast<uint4*>(dst);

  if (kFast) {
    double fs = 0.0;
    uint32_t umin = 0xffffffffu, umax = 0u;
    for (int c = threadIdx.x; c < 2 * n16; c += kNormThreads) {
      const uint4 hv = __ldg(src4 + c);
      const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t ul = (w[j] & 0x7fffu) << 13, uh = (w[j] & 0x7fff0000u) >> 3;
        umin = min(umin, min(ul, uh));
        umax = max(umax, max(ul, uh));
        const double lo = __hiloint2double((int)(ul + 0x38000000u), 0);
        const double hi = __hiloint2double((int)(uh + 0x38000000u), 0);
        fs += lo * lo;
        fs += hi * hi;
      }
    }
#pragma unroll
    for (int m = 16; m; m >>= 1) {
      fs += __shfl_xor_sync(0xffffffffu, fs, m);
      umin = min(umin, __shfl_xor_sync(0xffffffffu, umin, m));
      umax = max(umax, __shfl_xor_sync(0xffffffffu, umax, m));
    }
    if (lane == 0) {
      s_ss[warp] = fs;
      s_mx[warp] = __uint_as_float(umax << 3);           // the pattern back in float position
      // exponent field 0 or 255 somewhere, or an element more than 2^40 below the peak (its
      // t' could leave the float range the encoder below works in)
      s_bad[warp] = (umin < 0x00100000u) | (umax >= 0x0ff00000u);
      s_lo[warp] = umin;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = 0.0;
      float peak = 0.f;
      int b = 0;
      uint32_t lo_all = 0xffffffffu;
      for (int w = 0; w < kNormThreads / 32; ++w) {
        tot += s_ss[w]; peak = fmaxf(peak, s_mx[w]); b |= s_bad[w]; lo_all = min(lo_all, s_lo[w]);
      }
      b |= ((__float_as_uint(peak) >> 23) - (lo_all >> 20)) >= 40u;
      if (!b) {
        const double inv = 1.0 / sqrt(tot);
        const float scale = (float)((double)peak * inv / 448.0);
        s_inv = inv;
        s_scale = scale;
        s_g = inv / (double)scale;
        *scale_out = scale;
      }
      s_ok = b ? -1 : 1;
    }
    __syncthreads();
    if (s_ok == 1) {
      const double inv = s_inv, sc = (double)s_scale, g = s_g;
      for (int c = threadIdx.x; c < n16; c += kNormThreads) {
        uint32_t o[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint4 hv = __ldg(src4 + 2 * c + h);
          const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
          uint32_t c16[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            // |x| of the word's two elements as doubles, times g
            const uint32_t hl = (w[j] & 0x7fffu) * 8192u + 0x38000000u;
            const uint32_t hh = __umulhi(w[j] & 0x7fff0000u, 0x20000000u) + 0x38000000u;
            const double t0 = __hiloint2double((int)hl, 0) * g;
            const double t1 = __hiloint2double((int)hh, 0) * g;
            const uint32_t a0 = (uint32_t)__double2hiint(t0), b0 = (uint32_t)__double2loint(t0);
            const uint32_t a1 = (uint32_t)__double2hiint(t1), b1 = (uint32_t)__double2loint(t1);
            // the same value as a float: exponent rebiased (by -896 << 23, modulo 2^32), the
            // 20 fraction bits of the high word, and a sticky last bit for the low word, so
            // that the hardware's round-to-nearest-even into E4M3 (subnormal codes and the
            // cap at 448 included) sees on which side of a boundary t' lies
            const float f0 = __uint_as_float(((a0 << 3) + 0x40000000u) | min(b0, 1u));
            const float f1 = __uint_as_float(((a1 << 3) + 0x40000000u) | min(b1, 1u));
            uint16_t two;
            asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(two) : "f"(f1), "f"(f0));
            uint32_t cd = two;
            const bool n0 = ((a0 + 1u) & 0x1fffeu) == 0x10000u;   // 0xffff or 0x10000:
            const bool n1 = ((a1 + 1u) & 0x1fffeu) == 0x10000u;   // the low word decides
            if (n0 | n1) {
              if (n0 && ((a0 & 1u) ? b0 >= 0xffffff00u : b0 < 0x100u))
                cd = (cd & 0xff00u) | (e4m3_encode_element(bf16_lo(w[j]), inv, sc) & 0x7fu);
              if (n1 && ((a1 & 1u) ? b1 >= 0xffffff00u : b1 < 0x100u))
                cd = (cd & 0x00ffu) | ((e4m3_encode_element(bf16_hi(w[j]), inv, sc) & 0x7fu) << 8);
            }
            c16[j] = cd;
          }
          // four codes per word, then the four sign bits (bit 15 and 31 of each input word)
          o[2 * h] = (c16[0] | (c16[1] << 16)) | (__byte_perm(w[0], w[1], 0x7531) & 0x80808080u);
          o[2 * h + 1] = (c16[2] | (c16[3] << 16)) | (__byte_perm(w[2], w[3], 0x7531) & 0x80808080u);
        }
        dst4[c] = make_uint4(o[0], o[1], o[2], o[3]);
      }
      __syncthreads();   // the shared scratch is reused by the next row
      return true;
    }
  }

  double ss = 0.0;
  float mx = 0.f;
  int bad = 0;
  for (int c = threadIdx.x; c < 2 * n16; c += kNormThreads) {
    const uint4 hv = __ldg(src4 + c);
    const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float lo = bf16_lo(w[j]), hi = bf16_hi(w[j]);
      bad |= ((w[j] & 0x7f80u) == 0x7f80u) | ((w[j] & 0x7f800000u) == 0x7f800000u);
      ss += (double)lo * (double)lo;
      ss += (double)hi * (double)hi;
      mx = fmaxf(mx, fmaxf(fabsf(lo), fabsf(hi)));
    }
  }
#pragma unroll
  for (int m = 16; m; m >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, m);
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, m));
    bad |= __shfl_xor_sync(0xffffffffu, bad, m);
  }
  if (lane == 0) { s_ss[warp] = ss; s_mx[warp] = mx; s_bad[warp] = bad; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    float peak = 0.f;
    int b = 0;
    for (int w = 0; w < kNormThreads / 32; ++w) { tot += s_ss[w]; peak = fmaxf(peak, s_mx[w]); b |= s_bad[w]; }
    const double nrm = sqrt(tot);
    const bool ok = !b && nrm > 0.0 && isfinite(nrm);
    const double inv = ok ? 1.0 / nrm : 0.0;
    s_inv = inv;
    s_scale = ok ? (float)((double)peak * inv / 448.0) : 0.f;
    s_ok = ok ? 1 : 0;
    *scale_out = s_scale;
  }
  __syncthreads();
  const double inv = s_inv, sc = (double)s_scale;
  for (int c = threadIdx.x; c < n16; c += kNormThreads) {
    uint32_t o[4] = {0, 0, 0, 0};
    if (sc != 0.0) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint4 hv = __ldg(src4 + 2 * c + h);
        const uint32_t w[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t c0 = e4m3_encode(((double)bf16_lo(w[j]) * inv) / sc);
          const uint32_t c1 = e4m3_encode(((double)bf16_hi(w[j]) * inv) / sc);
          const int e = h * 8 + j * 2;                       // element index within the 16
          o[e >> 2] |= (c0 << ((e & 3) * 8)) | (c1 << (((e + 1) & 3) * 8));
        }
      }
    }
    dst4[c] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  const bool ok = s_ok != 0;
  __syncthreads();   // the shared scratch is reused by the next row
  return ok;
}

// One CTA per row.
__global__ void __launch_bounds__(kNormThreads, 4)
append_e4m3_kernel(const uint16_t* __restrict__ states, const int32_t* __restrict__ tokens,
                   int64_t n, int d, uint8_t* __restrict__ codes, float* __restrict__ scales,
                   int32_t* __restrict__ tok, int32_t* __restrict__ trace_id, int64_t row0,
                   int32_t trace, int32_t* __restrict__ trace_end,
                   uint64_t* __restrict__ trace_tag, uint64_t tag,
                   int64_t* __restrict__ trace_gbase, int64_t gbase, int set_tag,
                   DeviceStats* stats) {
  pdl_launch_dependents();
  pdl_wait();   // earlier queries may still be reading the trace table and token stream
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    trace_end[trace] = (int32_t)(row0 + n);
    if (set_tag) { trace_tag[trace] = tag; trace_gbase[trace] = gbase; }
  }
  for (int64_t r = blockIdx.x; r < n; r += gridDim.x) {
    const int64_t row = row0 + r;
    const bool ok = quantize_row_e4m3<true>(states + r * d, d, codes + row * d, scales + row);
    if (threadIdx.x == 0) {
      tok[row] = tokens[r];
      trace_id[row] = trace;
      if (!ok) atomicAdd(&stats->degenerate_rows, 1ull);           // stored as a zero key
    }
  }
}

cudaError_t launch_append_e4m3(const uint16_t* states, const int32_t* tokens, int64_t n, int32_t d,
                               uint8_t* codes, float* scales, int32_t* tok, int32_t* trace_id,
                               int64_t row0, int32_t trace, int32_t* trace_end,
                               uint64_t* trace_tag, uint64_t tag, int64_t* trace_gbase,
                               int64_t gbase, int set_tag, DeviceStats* stats, cudaStream_t st) {
  int64_t grid = n < 1 ? 1 : (n > 65535 * 8 ? 65535 * 8 : n);
  return launch_pdl(append_e4m3_kernel, dim3((unsigned)grid), dim3(kNormThreads), 0, st, states,
                    tokens, n, d, codes, scales, tok, trace_id, row0, trace, trace_end, trace_tag,
                    tag, trace_gbase, gbase, set_tag, stats);
}

// ----------------------------------------------------------------------- scan ---
constexpr int kQ8Threads = kNormThreads;
constexpr int kQ8Warps = kQ8Threads / 32;
constexpr int kQ8Rows = 4;        // rows a warp scores together

// two E4M3 codes -> two floats (exact)
__device__ __forceinline__ float2 e4m3x2_to_float2(uint32_t two_codes) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)two_codes));
  return __half22float2(*reinterpret_cast<const __half2*>(&h2));
}

// Same structure as the 16-bit CUDA-core scan: 2 CTAs x 8 warps per SM, contiguous row
// split, 16-byte streaming loads (16 codes), the normalised bf16 queries in shared memory,
// fp32 accumulation, per-warp sorted register lists, one list per CTA and query.
template <int QT, int E>
__global__ void __launch_bounds__(kQ8Threads, 2)
scan_gemv_e4m3_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scales,
                      PoolView pv, const uint16_t* __restrict__ q_raw, int nq, int k,
                      const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                      int32_t* __restrict__ q_valid, DeviceStats* stats, FusedAppend fa) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int KK = 32 * E;
  pdl_launch_dependents();
  pdl_wait();
  const int d = pv.d, n8 = d >> 3, n16 = d >> 4;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                        // [QT][n8] bf16
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)QT * d * 2);   // [warps][KK]
  __shared__ uint64_t s_ex[QT];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // contiguous, balanced share of the rows; the fa.n CTAs that first append a row of this
  // step take 1/16 less (quantising a row costs about twice what normalising one does)
  const int64_t n = pv.n_rows;
  const int64_t w_lo = 16ll * blockIdx.x - min((int)blockIdx.x, fa.n);
  const int64_t w_hi = 16ll * (blockIdx.x + 1) - min((int)blockIdx.x + 1, fa.n);
  const int64_t w_all = 16ll * gridDim.x - min((int)gridDim.x, fa.n);
  const int r_lo = (int)((n * w_lo) / w_all);
  const int r_hi = (int)((n * w_hi) / w_all);
  const uint4* codes4 = reinterpret_cast<const uint4*>(codes);

  // the step's append, one row per CTA (as in the 16-bit scan)
  if ((int)blockIdx.x < fa.n) {
    const int r = blockIdx.x;
    const int64_t row = (int64_t)fa.row0 + r;
    const bool ok = quantize_row_e4m3<true>(fa.states + (size_t)r * d, d,
                                      const_cast<uint8_t*>(codes) + row * d,
                                      const_cast<float*>(scales) + row);
    if (threadIdx.x == 0) {
      fa.tok[row] = fa.tokens[r];
      fa.trace_id[row] = fa.trace;
      if (!ok) atomicAdd(&stats->degenerate_rows, 1ull);
      if (r == 0) {
        fa.trace_end[fa.trace] = fa.row0 + fa.n;
        if (fa.set_tag) { fa.trace_tag[fa.trace] = fa.tag; fa.trace_gbase[fa.trace] = fa.gbase; }
      }
    }
    __threadfence();                   // this thread's part of the row, before the count
    __syncthreads();
    if (threadIdx.x == 0) {
      __threadfence();                 // cumulative: the whole CTA's row, as seen through the barrier
      atomicAdd(fa.ready, 1ull);
    }
  }
  bool fresh_ok = fa.n == 0;           // this warp has seen the appended rows arrive

  for (int q0 = 0; q0 < nq; q0 += QT) {
    __syncthreads();
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      uint16_t* dst = reinterpret_cast<uint16_t*>(qs + (size_t)q * n8);
      if (q0 + q < nq) {
        const int code = normalize_row<false>(q_raw + (size_t)(q0 + q) * d, dst, d);
        if (blockIdx.x == 0 && threadIdx.x == 0) {
          q_valid[q0 + q] = code == kRowNonFinite ? 0 : 1;
          if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
        }
      } else {
        for (int c = threadIdx.x; c < n8; c += kQ8Threads) qs[(size_t)q * n8 + c] = make_uint4(0, 0, 0, 0);
      }
    }
    if (threadIdx.x < QT)
      s_ex[threadIdx.x] = (exclude_tag && q0 + threadIdx.x < nq) ? exclude_tag[q0 + threadIdx.x] : 0;
    __syncthreads();

    u64 top[QT][E];
    u64 kth[QT];
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      kth[q] = 0;
#pragma unroll
      for (int r = 0; r < E; ++r) top[q][r] = 0;
    }

    for (int rb = r_lo + warp * kQ8Rows; rb < r_hi; rb += kQ8Warps * kQ8Rows) {
      const uint4* rowp[kQ8Rows];
#pragma unroll
      for (int r = 0; r < kQ8Rows; ++r) {
        const int row = rb + r < r_hi ? rb + r : r_hi - 1;      // clamp: result discarded below
        rowp[r] = codes4 + (size_t)row * n16;
      }
      float acc[kQ8Rows][QT];
#pragma unroll
      for (int r = 0; r < kQ8Rows; ++r)
#pragma unroll
        for (int q = 0; q < QT; ++q) acc[r][q] = 0.f;

      const bool fresh = fa.n > 0 && rb + kQ8Rows > fa.row0;       // warp-uniform
      if (fresh && !fresh_ok) {
        wait_fused_rows(fa, stats);       // rows of this step's append
        fresh_ok = true;
      }
#pragma unroll 4
      for (int c = lane; c < n16; c += 32) {
        uint4 kv[kQ8Rows];
#pragma unroll
        for (int r = 0; r < kQ8Rows; ++r)
          kv[r] = fresh ? ld_cg16(rowp[r] + c) : ld_stream16(rowp[r] + c);
        uint4 qv[QT][2];
#pragma unroll
        for (int q = 0; q < QT; ++q) { qv[q][0] = qs[q * n8 + 2 * c]; qv[q][1] = qs[q * n8 + 2 * c + 1]; }
#pragma unroll
        for (int j = 0; j < 4; ++j) {                     // word j of the 16 bytes: 4 codes
          float2 ka[kQ8Rows], kb[kQ8Rows];
#pragma unroll
          for (int r = 0; r < kQ8Rows; ++r) {
            const uint32_t w = j == 0 ? kv[r].x : (j == 1 ? kv[r].y : (j == 2 ? kv[r].z : kv[r].w));
            ka[r] = e4m3x2_to_float2(w & 0xffffu);
            kb[r] = e4m3x2_to_float2(w >> 16);
          }
#pragma unroll
          for (int q = 0; q < QT; ++q) {
            // elements 4j..4j+3 of the chunk: query words 2j and 2j+1 of its 8
            const uint4 h = qv[q][j >> 1];
            const uint32_t w0 = (j & 1) ? h.z : h.x, w1 = (j & 1) ? h.w : h.y;
            const float q0f = bf16_lo(w0), q1f = bf16_hi(w0), q2f = bf16_lo(w1), q3f = bf16_hi(w1);
#pragma unroll
            for (int r = 0; r < kQ8Rows; ++r) {
              float a = acc[r][q];
              a = fmaf(ka[r].x, q0f, a);
              a = fmaf(ka[r].y, q1f, a);
              a = fmaf(kb[r].x, q2f, a);
              a = fmaf(kb[r].y, q3f, a);
              acc[r][q] = a;
            }
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kQ8Rows; ++r) {
        const int row = rb + r;
        if (row >= r_hi) break;                             // warp-uniform
        const bool fresh_row = fa.n > 0 && row >= fa.row0;     // written by another CTA just now
        const float sc = fresh_row ? __ldcg(scales + row) : scales[row];
        uint64_t tag = 0;
        if (exclude_tag)
          tag = fresh_row ? __ldcg(&pv.trace_tag[__ldcg(&pv.trace_id[row])])
                          : pv.trace_tag[pv.trace_id[row]];
#pragma unroll
        for (int q = 0; q < QT; ++q) {
          const float s = warp_sum(acc[r][q]) * sc;
          if (q0 + q >= nq) continue;
          if (s_ex[q] != 0 && tag == s_ex[q]) continue;     // same-prompt trace: skipped
          const u64 key = pack_candidate(s, (uint32_t)row);
          if (key > kth[q]) {
            warp_sorted_insert<E>(top[q], key, lane);
            kth[q] = warp_list_get<E>(top[q], k - 1);
          }
        }
      }
    }
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      if (q0 + q >= nq) break;
      block_merge_desc<E>(top[q], scratch, kQ8Warps);
      if (threadIdx.x < 32) {
        u64* dst = partial + ((size_t)blockIdx.x * nq + (q0 + q)) * KK;
#pragma unroll
        for (int r = 0; r < E; ++r) dst[r * 32 + lane] = top[q][r];
      }
    }
  }
}

template <int QT, int E>
static cudaError_t launch_q8(const uint8_t* codes, const float* scales, const PoolView& pv,
                             const uint16_t* q_raw, int nq, int k, const uint64_t* ex, u64* partial,
                             int32_t* q_valid, DeviceStats* stats, int grid, const FusedAppend& fa,
                             cudaStream_t st) {
  const size_t smem = (size_t)QT * pv.d * 2 + (size_t)kQ8Warps * 32 * E * sizeof(u64);
  cudaError_t e = cudaFuncSetAttribute(scan_gemv_e4m3_kernel<QT, E>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(scan_gemv_e4m3_kernel<QT, E>, dim3(grid), dim3(kQ8Threads), smem, st, codes,
                    scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, fa);
}

template <int QT>
static cudaError_t launch_q8_qt(int kk, const uint8_t* codes, const float* scales,
                                const PoolView& pv, const uint16_t* q_raw, int nq, int k,
                                const uint64_t* ex, u64* partial, int32_t* q_valid,
                                DeviceStats* stats, int grid, const FusedAppend& fa,
                                cudaStream_t st) {
  if (kk == 32) return launch_q8<QT, 1>(codes, scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
  if (kk == 64) return launch_q8<QT, 2>(codes, scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
  return launch_q8<QT, 4>(codes, scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
}

cudaError_t launch_scan_gemv_e4m3(const uint8_t* codes, const float* scales, const PoolView& pv,
                                  const uint16_t* q_raw, int32_t nq, int32_t k, int32_t kk,
                                  const uint64_t* exclude_tag, unsigned long long* partial,
                                  int32_t* q_valid, DeviceStats* stats, int32_t max_lists,
                                  int32_t num_sms, int32_t* n_lists, const FusedAppend* fused,
                                  cudaStream_t st) {
  const int grid = scan_gemv_grid(pv.n_rows, num_sms, max_lists);
  *n_lists = grid;
  FusedAppend fa = {};
  if (fused) {
    if (fused->n > grid || fused->n > kFuseMaxRows) return cudaErrorInvalidValue;
    fa = *fused;
  }
  if (nq >= 2)
    return launch_q8_qt<2>(kk, codes, scales, pv, q_raw, nq, k, exclude_tag, partial, q_valid, stats, grid, fa, st);
  return launch_q8_qt<1>(kk, codes, scales, pv, q_raw, nq, k, exclude_tag, partial, q_valid, stats, grid, fa, st);
}

}  // namespace oilbird
