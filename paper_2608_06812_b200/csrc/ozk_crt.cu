// Reconstruction kernel (Section 5.2: single-pass direct CRT in integer arithmetic;
// Section 4.2: inverse scaling and one rounding to FP64).
//
// Per output element:  S = sum_l r_l w_l  (multiword, 32-bit limbs)
//                      q ~ S / P in FP64, x = S - q P, corrected into [0, P)
//                      x -> x - P if x > P/2
//                      C = RN_even(x * 2^-(s_i + t_j))
// Everything is column-major with the row index fastest, so one thread per element
// coalesces the residue bytes, the shifts and the FP64 stores alike.
#include "ozk_common.cuh"
#include "ozk_round.cuh"

namespace ozk {
namespace {

template <int NW>
__global__ void __launch_bounds__(256) crt_kernel(CrtTable ct, const uint8_t* __restrict__ res, int64_t res_ld,
                                                  size_t res_stride, const int32_t* __restrict__ s,
                                                  const int32_t* __restrict__ t, int64_t M, double* __restrict__ C,
                                                  int64_t ldc, uint32_t* __restrict__ x_out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t j = blockIdx.y;
  if (i >= M) return;
  const uint8_t* rp = res + (size_t)j * (size_t)res_ld + (size_t)i;
  uint32_t S[NW];
#pragma unroll
  for (int k = 0; k < NW; ++k) S[k] = 0;
  for (int l = 0; l < ct.L; ++l) {
    const uint32_t r = rp[(size_t)l * res_stride];
    uint32_t carry = 0;
#pragma unroll
    for (int k = 0; k < NW; ++k) {
      const uint64_t v = (uint64_t)r * ct.w[l][k] + S[k] + carry;
      S[k] = (uint32_t)v;
      carry = (uint32_t)(v >> 32);
    }
  }
  // quotient estimate in FP64, then exact correction
  double Sd = 0.0;
#pragma unroll
  for (int k = NW - 1; k >= 0; --k) Sd = Sd * 4294967296.0 + (double)S[k];
  const uint32_t q = (uint32_t)(Sd * ct.inv_P);
  {
    uint32_t borrow = 0, carry = 0;  // S -= q * P, two's complement over NW words plus a sign word
    uint32_t signw = 0;
#pragma unroll
    for (int k = 0; k < NW; ++k) {
      const uint64_t prod = (uint64_t)q * ct.P[k] + carry;
      carry = (uint32_t)(prod >> 32);
      const uint64_t d = (uint64_t)S[k] - (uint32_t)prod - borrow;
      S[k] = (uint32_t)d;
      borrow = (uint32_t)(d >> 63);
    }
    signw = 0u - carry - borrow;  // 0 if non-negative, all ones if the estimate overshot
#pragma unroll 1
    for (int it = 0; it < 2 && signw != 0; ++it) {  // negative: add P back
      uint32_t c2 = 0;
#pragma unroll
      for (int k = 0; k < NW; ++k) {
        const uint64_t v = (uint64_t)S[k] + ct.P[k] + c2;
        S[k] = (uint32_t)v;
        c2 = (uint32_t)(v >> 32);
      }
      signw += c2;
    }
#pragma unroll 1
    for (int it = 0; it < 2 && ge<NW>(S, ct.P); ++it) sub_in_place<NW>(S, ct.P);
  }
  // symmetric representative
  bool neg = false;
  if (gt<NW>(S, ct.halfP)) {
    uint32_t tmp[NW];
#pragma unroll
    for (int k = 0; k < NW; ++k) tmp[k] = ct.P[k];
    sub_in_place<NW>(tmp, S);
#pragma unroll
    for (int k = 0; k < NW; ++k) S[k] = tmp[k];
    neg = true;
  }
  const double mag = round_scaled<NW>(S, s[i] + t[j]);
  C[i + j * ldc] = neg ? -mag : mag;
  if (x_out) {
    uint32_t* xo = x_out + (size_t)kCrtWords * ((size_t)i + (size_t)j * (size_t)M);
    uint32_t carry = neg ? 1u : 0u;
#pragma unroll
    for (int k = 0; k < kCrtWords; ++k) {
      uint32_t w = k < NW ? S[k] : 0u;
      if (neg) {
        const uint64_t v = (uint64_t)(~w) + carry;
        w = (uint32_t)v;
        carry = (uint32_t)(v >> 32);
      }
      xo[k] = w;
    }
  }
}


// ------------------------------------------------------------------------------------
// Fast variant for aligned inputs: one thread reconstructs four consecutive rows i of one column j.
//   * residues come in as one 32-bit load per modulus (four bytes = four rows)
//   * S = sum r_l w_l is accumulated limb by limb in independent 64-bit sums (r < 2^8, w limb < 2^32,
//     at most 27 terms: no carries until the end), one multiply-add per (modulus, limb)
//   * the rounding builds the FP64 bit pattern directly (normalise, 53 bits, round bit, sticky); a
//     result in the subnormal range takes the general routine above
// ------------------------------------------------------------------------------------
template <int NW>
__device__ __forceinline__ double round_scaled_fast(const uint32_t (&mag)[NW], int shift) {
  // top non-zero word and the two words below it
  int top = -1;
#pragma unroll
  for (int i = 0; i < NW; ++i)
    if (mag[i]) top = i;
  if (top < 0) return 0.0;
  uint32_t w2 = 0, w1 = 0, w0 = 0, rest = 0;
#pragma unroll
  for (int i = 0; i < NW; ++i) {
    if (i == top) w2 = mag[i];
    if (i == top - 1) w1 = mag[i];
    if (i == top - 2) w0 = mag[i];
    if (i < top - 2) rest |= mag[i];
  }
  const int lz = __clz(w2);
  const int bitlen = 32 * top + 32 - lz;
  const int e_out = bitlen - 1 - shift;  // value in [2^e_out, 2^(e_out+1))
  if (e_out < -1022 || e_out > 1023) return round_scaled<NW>(mag, shift);  // subnormal or overflowing: general path
  // 64-bit window with the value's top bit at bit 63: the top 64 bits of (w2:w1:w0) << lz
  const uint32_t h1 = __funnelshift_l(w1, w2, lz), h0 = __funnelshift_l(w0, w1, lz);
  const unsigned long long h = ((unsigned long long)h1 << 32) | h0;
  const uint32_t below = (w0 << lz) | rest;  // everything under the window (for lz = 0 all of w0)
  unsigned long long mant = h >> 11;         // 53 bits, leading one at bit 52
  const bool round_bit = ((h >> 10) & 1ull) != 0ull;
  const bool sticky = ((h & 0x3FFull) != 0ull) || (below != 0u);
  if (round_bit && (sticky || (mant & 1ull))) ++mant;
  // exponent field and mantissa in one addition: the leading one adds 1 to the exponent field, and a
  // carry out of the mantissa (mant = 2^53) moves the result to the next binade (or to infinity)
  return __longlong_as_double((long long)(((unsigned long long)(e_out + 1022) << 52) + mant));
}


// Lean reconstruction for 2^100 <= P < 2^126 (16 to 19 moduli): the weighted sum S (five words)
// arrives as four 64-bit column sums; everything after the quotient estimate is 128-bit arithmetic
// written as explicit carry chains.
//   q  = floor((S >> 96) * (2^96 / P) * (1 - 2^-30))  is the true quotient or one below it, so
//   x  = S - q P  lies in [0, 2P) and fits 128 bits; one conditional subtraction brings it below P.
__device__ __forceinline__ double reconstruct_lean(const unsigned long long (&acc)[4], const CrtTable& ct, int shift) {
  const uint32_t a0l = (uint32_t)acc[0], a0h = (uint32_t)(acc[0] >> 32), a1l = (uint32_t)acc[1], a1h = (uint32_t)(acc[1] >> 32);
  const uint32_t a2l = (uint32_t)acc[2], a2h = (uint32_t)(acc[2] >> 32), a3l = (uint32_t)acc[3], a3h = (uint32_t)(acc[3] >> 32);
  uint32_t S1, S2, S3, S4;
  asm("add.cc.u32 %0, %4, %5;\n\t"
      "addc.cc.u32 %1, %6, %7;\n\t"
      "addc.cc.u32 %2, %8, %9;\n\t"
      "addc.u32 %3, %10, 0;"
      : "=r"(S1), "=r"(S2), "=r"(S3), "=r"(S4)
      : "r"(a0h), "r"(a1l), "r"(a1h), "r"(a2l), "r"(a2h), "r"(a3l), "r"(a3h));
  const uint32_t S0 = a0l;
  const unsigned long long top = ((unsigned long long)S4 << 32) | S3;
  const uint32_t q = __double2uint_rz(__ull2double_rz(top) * ct.q_scale);
  const unsigned long long m0 = (unsigned long long)q * ct.P[0];
  const unsigned long long m1 = (unsigned long long)q * ct.P[1] + (m0 >> 32);
  const unsigned long long m2 = (unsigned long long)q * ct.P[2] + (m1 >> 32);
  const unsigned long long m3 = (unsigned long long)q * ct.P[3] + (m2 >> 32);
  uint32_t x0, x1, x2, x3;
  asm("sub.cc.u32 %0, %4, %8;\n\t"
      "subc.cc.u32 %1, %5, %9;\n\t"
      "subc.cc.u32 %2, %6, %10;\n\t"
      "subc.u32 %3, %7, %11;"
      : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3)
      : "r"(S0), "r"(S1), "r"(S2), "r"(S3), "r"((uint32_t)m0), "r"((uint32_t)m1), "r"((uint32_t)m2), "r"((uint32_t)m3));
  const uint32_t P0 = ct.P[0], P1 = ct.P[1], P2 = ct.P[2], P3 = ct.P[3];
  uint32_t d0, d1, d2, d3, below;  // d = x - P; below = all ones if x < P
  asm("sub.cc.u32 %0, %5, %9;\n\t"
      "subc.cc.u32 %1, %6, %10;\n\t"
      "subc.cc.u32 %2, %7, %11;\n\t"
      "subc.cc.u32 %3, %8, %12;\n\t"
      "subc.u32 %4, 0, 0;"
      : "=r"(d0), "=r"(d1), "=r"(d2), "=r"(d3), "=r"(below)
      : "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(P0), "r"(P1), "r"(P2), "r"(P3));
  if (!below) x0 = d0, x1 = d1, x2 = d2, x3 = d3;
  uint32_t e0, e1, e2, e3;  // e = P - x
  asm("sub.cc.u32 %0, %4, %8;\n\t"
      "subc.cc.u32 %1, %5, %9;\n\t"
      "subc.cc.u32 %2, %6, %10;\n\t"
      "subc.u32 %3, %7, %11;"
      : "=r"(e0), "=r"(e1), "=r"(e2), "=r"(e3)
      : "r"(P0), "r"(P1), "r"(P2), "r"(P3), "r"(x0), "r"(x1), "r"(x2), "r"(x3));
  uint32_t u0, u1, u2, u3, over;  // halfP - x borrows exactly when x > P/2
  asm("sub.cc.u32 %0, %5, %9;\n\t"
      "subc.cc.u32 %1, %6, %10;\n\t"
      "subc.cc.u32 %2, %7, %11;\n\t"
      "subc.cc.u32 %3, %8, %12;\n\t"
      "subc.u32 %4, 0, 0;"
      : "=r"(u0), "=r"(u1), "=r"(u2), "=r"(u3), "=r"(over)
      : "r"(ct.halfP[0]), "r"(ct.halfP[1]), "r"(ct.halfP[2]), "r"(ct.halfP[3]), "r"(x0), "r"(x1), "r"(x2), "r"(x3));
  uint32_t mag[4];
  mag[0] = over ? e0 : x0;
  mag[1] = over ? e1 : x1;
  mag[2] = over ? e2 : x2;
  mag[3] = over ? e3 : x3;
  const double r = round_scaled_fast<4>(mag, shift);
  return over ? -r : r;
}

// The same for 2^128 <= P < 2^158 (20 to 23 moduli): S has six words and arrives as five 64-bit column sums,
// the quotient estimate uses the words above bit 128 (q_scale128 = (2^128 / P)(1 - 2^-30); the part of S below
// bit 128 is less than P, so the estimate is again the true quotient or one below it), x has five words.
__device__ __forceinline__ double reconstruct_lean5(const unsigned long long (&acc)[5], const CrtTable& ct, int shift) {
  const uint32_t a0l = (uint32_t)acc[0], a0h = (uint32_t)(acc[0] >> 32), a1l = (uint32_t)acc[1], a1h = (uint32_t)(acc[1] >> 32);
  const uint32_t a2l = (uint32_t)acc[2], a2h = (uint32_t)(acc[2] >> 32), a3l = (uint32_t)acc[3], a3h = (uint32_t)(acc[3] >> 32);
  const uint32_t a4l = (uint32_t)acc[4], a4h = (uint32_t)(acc[4] >> 32);
  uint32_t S1, S2, S3, S4, S5;
  asm("add.cc.u32 %0, %5, %6;\n\t"
      "addc.cc.u32 %1, %7, %8;\n\t"
      "addc.cc.u32 %2, %9, %10;\n\t"
      "addc.cc.u32 %3, %11, %12;\n\t"
      "addc.u32 %4, %13, 0;"
      : "=r"(S1), "=r"(S2), "=r"(S3), "=r"(S4), "=r"(S5)
      : "r"(a0h), "r"(a1l), "r"(a1h), "r"(a2l), "r"(a2h), "r"(a3l), "r"(a3h), "r"(a4l), "r"(a4h));
  const uint32_t S0 = a0l;
  const unsigned long long top = ((unsigned long long)S5 << 32) | S4;
  const uint32_t q = __double2uint_rz(__ull2double_rz(top) * ct.q_scale128);
  const unsigned long long m0 = (unsigned long long)q * ct.P[0];
  const unsigned long long m1 = (unsigned long long)q * ct.P[1] + (m0 >> 32);
  const unsigned long long m2 = (unsigned long long)q * ct.P[2] + (m1 >> 32);
  const unsigned long long m3 = (unsigned long long)q * ct.P[3] + (m2 >> 32);
  const unsigned long long m4 = (unsigned long long)q * ct.P[4] + (m3 >> 32);
  uint32_t x0, x1, x2, x3, x4;
  asm("sub.cc.u32 %0, %5, %10;\n\t"
      "subc.cc.u32 %1, %6, %11;\n\t"
      "subc.cc.u32 %2, %7, %12;\n\t"
      "subc.cc.u32 %3, %8, %13;\n\t"
      "subc.u32 %4, %9, %14;"
      : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3), "=r"(x4)
      : "r"(S0), "r"(S1), "r"(S2), "r"(S3), "r"(S4), "r"((uint32_t)m0), "r"((uint32_t)m1), "r"((uint32_t)m2), "r"((uint32_t)m3),
        "r"((uint32_t)m4));
  const uint32_t P0 = ct.P[0], P1 = ct.P[1], P2 = ct.P[2], P3 = ct.P[3], P4 = ct.P[4];
  uint32_t d0, d1, d2, d3, d4, below;  // d = x - P; below = all ones if x < P
  asm("sub.cc.u32 %0, %6, %11;\n\t"
      "subc.cc.u32 %1, %7, %12;\n\t"
      "subc.cc.u32 %2, %8, %13;\n\t"
      "subc.cc.u32 %3, %9, %14;\n\t"
      "subc.cc.u32 %4, %10, %15;\n\t"
      "subc.u32 %5, 0, 0;"
      : "=r"(d0), "=r"(d1), "=r"(d2), "=r"(d3), "=r"(d4), "=r"(below)
      : "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(x4), "r"(P0), "r"(P1), "r"(P2), "r"(P3), "r"(P4));
  if (!below) x0 = d0, x1 = d1, x2 = d2, x3 = d3, x4 = d4;
  uint32_t e0, e1, e2, e3, e4;  // e = P - x
  asm("sub.cc.u32 %0, %5, %10;\n\t"
      "subc.cc.u32 %1, %6, %11;\n\t"
      "subc.cc.u32 %2, %7, %12;\n\t"
      "subc.cc.u32 %3, %8, %13;\n\t"
      "subc.u32 %4, %9, %14;"
      : "=r"(e0), "=r"(e1), "=r"(e2), "=r"(e3), "=r"(e4)
      : "r"(P0), "r"(P1), "r"(P2), "r"(P3), "r"(P4), "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(x4));
  uint32_t u0, u1, u2, u3, u4, over;  // halfP - x borrows exactly when x > P/2
  asm("sub.cc.u32 %0, %6, %11;\n\t"
      "subc.cc.u32 %1, %7, %12;\n\t"
      "subc.cc.u32 %2, %8, %13;\n\t"
      "subc.cc.u32 %3, %9, %14;\n\t"
      "subc.cc.u32 %4, %10, %15;\n\t"
      "subc.u32 %5, 0, 0;"
      : "=r"(u0), "=r"(u1), "=r"(u2), "=r"(u3), "=r"(u4), "=r"(over)
      : "r"(ct.halfP[0]), "r"(ct.halfP[1]), "r"(ct.halfP[2]), "r"(ct.halfP[3]), "r"(ct.halfP[4]), "r"(x0), "r"(x1), "r"(x2), "r"(x3),
        "r"(x4));
  uint32_t mag[5];
  mag[0] = over ? e0 : x0;
  mag[1] = over ? e1 : x1;
  mag[2] = over ? e2 : x2;
  mag[3] = over ? e3 : x3;
  mag[4] = over ? e4 : x4;
  const double r = round_scaled_fast<5>(mag, shift);
  return over ? -r : r;
}

// LMAX bounds the unrolled loops over the moduli (iterations beyond ct.L are predicated off but still
// issue, so the common case of at most 19 moduli gets its own instantiation).
// EXACT: ct.L equals LMAX, no per-modulus guard at all.
template <int WW, int NW, int LEAN, int LMAX, bool EXACT = false>
__global__ void __launch_bounds__(256, LEAN ? 4 : 2) crt4_kernel(const __grid_constant__ CrtTable ct, const uint8_t* __restrict__ res,
                                                   int64_t res_ld, size_t res_stride, const int32_t* __restrict__ s,
                                                   const int32_t* __restrict__ t, int64_t M, int64_t N,
                                                   double* __restrict__ C, int64_t ldc) {
  const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= M) return;
  for (int64_t j = blockIdx.y; j < N; j += gridDim.y) {
    const uint8_t* rp = res + (size_t)j * (size_t)res_ld + (size_t)i;
    unsigned long long acc[4][WW];
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
      for (int k = 0; k < WW; ++k) acc[e][k] = 0ull;
    // all residue loads are issued before the first use: 19..27 independent 128-byte requests per
    // warp in flight instead of one (the streams of the moduli are 'res_stride' bytes apart)
    uint32_t r4[LMAX];
#pragma unroll
    for (int l = 0; l < LMAX; ++l)
      r4[l] = (EXACT || l < ct.L) ? __ldg(reinterpret_cast<const uint32_t*>(rp + (size_t)l * res_stride)) : 0u;
#pragma unroll
    for (int l = 0; l < LMAX; ++l) {
      if (EXACT || l < ct.L) {
#pragma unroll
        for (int k = 0; k < WW; ++k) {
          const uint32_t w = ct.w[l][k];
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[e][k] += (unsigned long long)__byte_perm(r4[l], 0u, 0x4440u + e) * w;
        }
      }
    }
    const int tj = t[j];
    const int4 s4 = *reinterpret_cast<const int4*>(s + i);
    const int sh[4] = {s4.x + tj, s4.y + tj, s4.z + tj, s4.w + tj};
    double out[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if constexpr (LEAN == 4) {
        static_assert(LEAN != 4 || (WW == 4 && NW == 5), "this lean tail is written for 4 weight words, 5 sum words");
        unsigned long long a4[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) a4[k] = acc[e][k < WW ? k : 0];
        out[e] = reconstruct_lean(a4, ct, sh[e]);
        continue;
      }
      if constexpr (LEAN == 5) {
        static_assert(LEAN != 5 || (WW == 5 && NW == 6), "this lean tail is written for 5 weight words, 6 sum words");
        unsigned long long a5[5];
#pragma unroll
        for (int k = 0; k < 5; ++k) a5[k] = acc[e][k < WW ? k : 0];
        out[e] = reconstruct_lean5(a5, ct, sh[e]);
        continue;
      }
      uint32_t S[NW];
      unsigned long long carry = 0ull;
#pragma unroll
      for (int k = 0; k < NW; ++k) {
        const unsigned long long v = (k < WW ? acc[e][k] : 0ull) + carry;
        S[k] = (uint32_t)v;
        carry = v >> 32;
      }
      // quotient estimate from the three top words (truncation error << 1), exact correction
      double Sd = (double)S[NW - 1];
      if (NW >= 2) Sd = Sd * 4294967296.0 + (double)S[NW - 2];
      if (NW >= 3) Sd = Sd * 4294967296.0 + (double)S[NW - 3];
      if (NW > 3) Sd *= __longlong_as_double((long long)(1023 + 32 * (NW - 3)) << 52);
      const uint32_t q = (uint32_t)(Sd * ct.inv_P);
      uint32_t borrow = 0, mc = 0;
#pragma unroll
      for (int k = 0; k < NW; ++k) {
        const unsigned long long prod = (unsigned long long)q * ct.P[k] + mc;
        mc = (uint32_t)(prod >> 32);
        const unsigned long long d = (unsigned long long)S[k] - (uint32_t)prod - borrow;
        S[k] = (uint32_t)d;
        borrow = (uint32_t)(d >> 63);
      }
      uint32_t signw = 0u - mc - borrow;
#pragma unroll 1
      for (int it = 0; it < 2 && signw != 0; ++it) {
        uint32_t c2 = 0;
#pragma unroll
        for (int k = 0; k < NW; ++k) {
          const unsigned long long v = (unsigned long long)S[k] + ct.P[k] + c2;
          S[k] = (uint32_t)v;
          c2 = (uint32_t)(v >> 32);
        }
        signw += c2;
      }
#pragma unroll 1
      for (int it = 0; it < 2 && ge<NW>(S, ct.P); ++it) sub_in_place<NW>(S, ct.P);
      bool neg = false;
      if (gt<NW>(S, ct.halfP)) {
        uint32_t tmp[NW];
#pragma unroll
        for (int k = 0; k < NW; ++k) tmp[k] = ct.P[k];
        sub_in_place<NW>(tmp, S);
#pragma unroll
        for (int k = 0; k < NW; ++k) S[k] = tmp[k];
        neg = true;
      }
      const double mag = round_scaled_fast<NW>(S, sh[e]);
      out[e] = neg ? -mag : mag;
    }
    double* dst = C + i + j * ldc;
    if (i + 4 <= M && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
      reinterpret_cast<double2*>(dst)[0] = make_double2(out[0], out[1]);
      reinterpret_cast<double2*>(dst)[1] = make_double2(out[2], out[3]);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (i + e < M) dst[e] = out[e];
    }
  }
}

__global__ void copy_residues_kernel(const uint8_t* __restrict__ res, int64_t Mp, size_t res_stride, int64_t M, int64_t N,
                                     uint8_t* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t j = blockIdx.y;
  const int64_t l = blockIdx.z;
  if (i >= M) return;
  out[(size_t)l * (size_t)M * (size_t)N + (size_t)j * (size_t)M + (size_t)i] =
      res[(size_t)l * res_stride + (size_t)j * (size_t)Mp + (size_t)i];
}

// acc = (acc + chunk) mod m for one modulus per blockIdx.y: sums the residues of two k ranges
// (Section 5.1: the residue of a sum is the sum of the residues).  16 bytes per thread.
__global__ void add_residues_kernel(uint8_t* __restrict__ acc, const uint8_t* __restrict__ chunk, size_t per_modulus,
                                    ModulusTable mt) {
  const size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v * 16 >= per_modulus) return;
  const uint32_t m = (uint32_t)mt.m[blockIdx.y];
  uint4* pa = reinterpret_cast<uint4*>(acc + (size_t)blockIdx.y * per_modulus) + v;
  const uint4 a = *pa;
  const uint4 b = *(reinterpret_cast<const uint4*>(chunk + (size_t)blockIdx.y * per_modulus) + v);
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
  uint32_t out[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    uint32_t word = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      uint32_t r = ((aw[k] >> (8 * e)) & 0xFFu) + ((bw[k] >> (8 * e)) & 0xFFu);
      r = min(r, r - m);
      word |= r << (8 * e);
    }
    out[k] = word;
  }
  *pa = make_uint4(out[0], out[1], out[2], out[3]);
}

}  // namespace

cudaError_t launch_add_residues(const Geometry& g, const ModulusTable& mt, uint8_t* acc, const uint8_t* chunk, cudaStream_t st) {
  const size_t per_modulus = (size_t)g.Mp * (size_t)g.Np;  // a multiple of 16
  dim3 grid((unsigned)((per_modulus / 16 + 255) / 256), (unsigned)g.L);
  add_residues_kernel<<<grid, 256, 0, st>>>(acc, chunk, per_modulus, mt);
  return cudaGetLastError();
}

cudaError_t launch_crt(const Geometry& g, const CrtTable& ct, const uint8_t* res, int64_t res_ld, size_t res_stride,
                       const int32_t* s, const int32_t* t, double* C, int64_t ldc, uint32_t* x_out, cudaStream_t st) {
  // weight words actually used, and whether the four-row kernel's vector loads are legal here
  int ww = 1;
  for (int l = 0; l < ct.L; ++l)
    for (int k = 0; k < kCrtWords; ++k)
      if (ct.w[l][k] && k + 1 > ww) ww = k + 1;
  const bool s_padded = (const void*)s == (const void*)(workspace_ptr() + g.off_s);  // the workspace copy has Mp entries
  const bool fast = !x_out && (res_ld % 4 == 0) && (res_stride % 4 == 0) && ((reinterpret_cast<uintptr_t>(res) & 3) == 0) &&
                    ((reinterpret_cast<uintptr_t>(s) & 15) == 0) && (g.M % 4 == 0 || s_padded);
  if (fast) {
    dim3 grid((unsigned)((g.M + 1023) / 1024), (unsigned)(g.N < 65535 ? g.N : 65535));
#define OZK_CRT4(WW, NW)                                                                                             \
  do {                                                                                                             \
    if (ct.L <= 19)                                                                                                \
      crt4_kernel<WW, NW, 0, 19><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc);   \
    else                                                                                                           \
      crt4_kernel<WW, NW, 0, kMaxModuli><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc); \
  } while (0)
    const bool lean = ct.words <= 5 && ww <= 4 && ct.p_bits >= 101 && ct.p_bits <= 126;  // 16 to 19 moduli
    const bool lean5 = ct.words <= 6 && ww <= 5 && ct.p_bits >= 129 && ct.p_bits <= 158;  // 20 to 23 moduli
#define OZK_CRT_LEAN5(LL) crt4_kernel<5, 6, 5, LL, true><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc)
    if (lean5 && ct.L == 20) OZK_CRT_LEAN5(20);
    else if (lean5 && ct.L == 21) OZK_CRT_LEAN5(21);
    else if (lean5 && ct.L == 22) OZK_CRT_LEAN5(22);
    else if (lean5 && ct.L == 23) OZK_CRT_LEAN5(23);
#undef OZK_CRT_LEAN5
    else
#define OZK_CRT_LEAN(LL) crt4_kernel<4, 5, 4, LL, true><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc)
    if (lean && ct.L == 19) OZK_CRT_LEAN(19);
    else if (lean && ct.L == 18) OZK_CRT_LEAN(18);
    else if (lean && ct.L == 17) OZK_CRT_LEAN(17);
    else if (lean && ct.L == 16) OZK_CRT_LEAN(16);
#undef OZK_CRT_LEAN
    else if (lean)
      crt4_kernel<4, 5, 4, 19><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc);
    else if (ct.words == 5 && ww <= 4) OZK_CRT4(4, 5);
    else if (ct.words <= 2) OZK_CRT4(2, 2);
    else if (ct.words == 3) OZK_CRT4(3, 3);
    else if (ct.words == 4) OZK_CRT4(4, 4);
    else if (ct.words == 5) OZK_CRT4(5, 5);
    else OZK_CRT4(6, 6);
#undef OZK_CRT4
    return cudaGetLastError();
  }
  dim3 grid((unsigned)((g.M + 255) / 256), (unsigned)g.N);
  switch (ct.words) {
    case 2: crt_kernel<2><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, C, ldc, x_out); break;
    case 3: crt_kernel<3><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, C, ldc, x_out); break;
    case 4: crt_kernel<4><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, C, ldc, x_out); break;
    case 5: crt_kernel<5><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, C, ldc, x_out); break;
    default: crt_kernel<6><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, C, ldc, x_out); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_copy_residues(const Geometry& g, const uint8_t* res, uint8_t* out, cudaStream_t st) {
  dim3 grid((unsigned)((g.M + 255) / 256), (unsigned)g.N, (unsigned)g.L);
  copy_residues_kernel<<<grid, 256, 0, st>>>(res, g.Mp, (size_t)g.Mp * (size_t)g.Np, g.M, g.N, out);
  return cudaGetLastError();
}

}  // namespace ozk
