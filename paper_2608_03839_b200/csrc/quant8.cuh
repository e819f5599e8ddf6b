// Row quantiser of pools with 8-bit keys (FP8 E4M3 codes + one fp32 scale per row), shared by
// the append kernel and by the scans that append a serving step's rows themselves.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"
#include "normalize.cuh"

namespace oilbird {

// two E4M3 codes -> two floats (exact)
__device__ __forceinline__ float2 e4m3x2_to_float2(uint32_t two_codes) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)two_codes));
  return __half22float2(*reinterpret_cast<const __half2*>(&h2));
}

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
static __device__ __noinline__ uint32_t e4m3_encode_element(float x, double inv, double sc) {
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
// kTid0 / kBar: the kNormThreads threads that take part are threads kTid0 .. kTid0 + 255 of
// the block, and they meet at named barrier kBar (0: they are the whole block).
template <bool kFast = false, int kTid0 = 0, int kBar = 0>
__device__ __forceinline__ bool quantize_row_e4m3(const uint16_t* __restrict__ src, int d,
                                                  uint8_t* __restrict__ dst, float* scale_out) {
  const int tid = (int)threadIdx.x - kTid0;
  auto sync = [] {
    if (kBar == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"n"(kBar), "n"(kNormThreads) : "memory");
  };
  __shared__ double s_ss[kNormThreads / 32];
  __shared__ float s_mx[kNormThreads / 32];
  __shared__ int s_bad[kNormThreads / 32];
  __shared__ uint32_t s_lo[kNormThreads / 32];
  __shared__ double s_inv;
  __shared__ double s_g;
  __shared__ float s_scale;
  __shared__ int s_ok;
  const int warp = tid >> 5, lane = tid & 31;
  const int n16 = d >> 4;
  const uint4* src4 = reinterpret_cast<const uint4*>(src);
  uint4* dst4 = reinterpret_cast<uint4*>(dst);

  if (kFast) {
    double fs = 0.0;
    uint32_t umin = 0xffffffffu, umax = 0u;
    for (int c = tid; c < 2 * n16; c += kNormThreads) {
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
    sync();
    if (tid == 0) {
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
    sync();
    if (s_ok == 1) {
      const double inv = s_inv, sc = (double)s_scale, g = s_g;
      for (int c = tid; c < n16; c += kNormThreads) {
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
      sync();   // the shared scratch is reused by the next row
      return true;
    }
  }

  double ss = 0.0;
  float mx = 0.f;
  int bad = 0;
  for (int c = tid; c < 2 * n16; c += kNormThreads) {
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
  sync();
  if (tid == 0) {
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
  sync();
  const double inv = s_inv, sc = (double)s_scale;
  for (int c = tid; c < n16; c += kNormThreads) {
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
  sync();   // the shared scratch is reused by the next row
  return ok;
}

}  // namespace oilbird
