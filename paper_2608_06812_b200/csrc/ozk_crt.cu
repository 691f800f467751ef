// Reconstruction kernel (Section 5.2: single-pass direct CRT in integer arithmetic;
// Section 4.2: inverse scaling and one rounding to FP64).
//
// Per output element:  S = sum_l r_l w_l  (multiword, 32-bit limbs)
//                      q ~ S / P in FP64, x = S - q P, corrected into [0, P)
//                      x -> x - P if x > P/2
//                      C = RN_even(x * 2^-(s_i + t_j))
// Everything is column-major with the row index fastest, so one thread per element
// coalesces the residue bytes, the shifts and the FP64 stores alike.
#include <algorithm>

#include "ozk_common.cuh"
#include "ozk_round.cuh"

namespace ozk {
namespace {

template <int NW>
__global__ void __launch_bounds__(256) crt_kernel(CrtTable ct, const uint8_t* __restrict__ res, int64_t res_ld,
                                                  size_t res_stride, const int32_t* __restrict__ s,
                                                  const int32_t* __restrict__ t, int64_t M, int64_t N,
                                                  double* __restrict__ C, int64_t ldc, uint32_t* __restrict__ x_out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  for (int64_t j = blockIdx.y; j < N; j += gridDim.y) {
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
  // top non-zero word and the two words below it; the usual case (top word in use) needs no search
  int top = NW - 1;
  uint32_t w2 = mag[NW - 1], w1 = NW >= 2 ? mag[NW >= 2 ? NW - 2 : 0] : 0u, w0 = NW >= 3 ? mag[NW >= 3 ? NW - 3 : 0] : 0u, rest = 0;
  if (w2 != 0) {
#pragma unroll
    for (int i = 0; i < NW - 3; ++i) rest |= mag[i];
  } else {
    top = -1;
#pragma unroll
    for (int i = 0; i < NW; ++i)
      if (mag[i]) top = i;
    if (top < 0) return 0.0;
    w2 = w1 = w0 = 0;
#pragma unroll
    for (int i = 0; i < NW; ++i) {
      if (i == top) w2 = mag[i];
      if (i == top - 1) w1 = mag[i];
      if (i == top - 2) w0 = mag[i];
      if (i < top - 2) rest |= mag[i];
    }
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


// Lean reconstruction for 2^84 <= P < 2^126 (13 to 19 moduli): the weighted sum S (up to 137 bits)
// arrives as four 64-bit column sums acc[k] (weight 2^(32 k), no carries yet).
//   q  = ((S >> (p_bits - 21)) * q_mul) >> 52 is the true quotient floor(S / P) or one below it.  The 32 bits
//        of S it needs come from the top column sums alone (from bit 96 up for P >= 2^116, where what is left out is
//        below 2^98 < P / 2^18; otherwise from bit 64 up with the carry out of the second sum, leaving out less than
//        2^66 < P / 2^18), which only lowers the estimate and keeps it in {floor(S / P) - 1, floor(S / P)}
//        (checked against big integers for every moduli count from 13 to 23, extreme residues included).
//   x  = S - q P in [0, 2P) is formed column by column as acc[k] + q n_k with n = 2^128 - P (one wide
//        multiply-add per word, then a single carry pass), modulo 2^128.
//   The two comparisons (x >= P, x > P / 2) look at the top word first; the full comparison runs only when
//   the top words are equal.  The rounding builds the FP64 bit pattern from the top three words directly;
//   a magnitude below 2^96 is moved one word up first; below 2^64, and results outside the normal range, take the
//   general routine.
__device__ __forceinline__ double reconstruct_lean(const unsigned long long (&acc)[4], const CrtTable& ct, int shift) {
  const uint32_t a3l = (uint32_t)acc[3], a3h = (uint32_t)(acc[3] >> 32), a2h = (uint32_t)(acc[2] >> 32);
  uint32_t t_lo, t_hi;
  asm("add.cc.u32 %0, %2, %4;\n\taddc.u32 %1, %3, 0;" : "=r"(t_lo), "=r"(t_hi) : "r"(a3l), "r"(a3h), "r"(a2h));
  uint32_t top;
  if (ct.q_word == 3) {
    top = __funnelshift_r(t_lo, t_hi, ct.q_bit);
  } else {
    const unsigned long long a64 = ((unsigned long long)t_hi << 32) | t_lo;
    const unsigned long long b64 = (a64 << 32) + (uint32_t)acc[2] + (acc[1] >> 32);
    top = (uint32_t)(b64 >> ct.q_bit);
  }
  const uint32_t q = __umulhi(top, ct.q_mul) >> 20;
  const uint32_t P0 = ct.P[0], P1 = ct.P[1], P2 = ct.P[2], P3 = ct.P[3];
  const unsigned long long c0 = acc[0] + (unsigned long long)q * ct.negP[0];  // negP = 2^128 - P
  const unsigned long long c1 = acc[1] + (unsigned long long)q * ct.negP[1];
  const unsigned long long c2 = acc[2] + (unsigned long long)q * ct.negP[2];
  const unsigned long long c3 = acc[3] + (unsigned long long)q * ct.negP[3];
  uint32_t x0 = (uint32_t)c0, x1, x2, x3;
  asm("add.cc.u32 %0, %3, %4;\n\taddc.cc.u32 %1, %5, %6;\n\taddc.u32 %2, %7, %8;"
      : "=r"(x1), "=r"(x2), "=r"(x3)
      : "r"((uint32_t)(c0 >> 32)), "r"((uint32_t)c1), "r"((uint32_t)(c1 >> 32)), "r"((uint32_t)c2), "r"((uint32_t)(c2 >> 32)), "r"((uint32_t)c3));
  if (x3 >= P3) {  // rarely true: x >= P needs the full comparison
    uint32_t d0, d1, d2, d3, below;
    asm("sub.cc.u32 %0, %5, %9;\n\tsubc.cc.u32 %1, %6, %10;\n\tsubc.cc.u32 %2, %7, %11;\n\tsubc.cc.u32 %3, %8, %12;\n\tsubc.u32 %4, 0, 0;"
        : "=r"(d0), "=r"(d1), "=r"(d2), "=r"(d3), "=r"(below)
        : "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(P0), "r"(P1), "r"(P2), "r"(P3));
    if (!below) x0 = d0, x1 = d1, x2 = d2, x3 = d3;
  }
  const uint32_t h3 = ct.halfP[3];
  bool over = x3 > h3;
  if (x3 == h3) {
    [[maybe_unused]] uint32_t u0, u1, u2, u3;  // only the borrow is wanted
    uint32_t bw;
    asm("sub.cc.u32 %0, %5, %9;\n\tsubc.cc.u32 %1, %6, %10;\n\tsubc.cc.u32 %2, %7, %11;\n\tsubc.cc.u32 %3, %8, %12;\n\tsubc.u32 %4, 0, 0;"
        : "=r"(u0), "=r"(u1), "=r"(u2), "=r"(u3), "=r"(bw)
        : "r"(ct.halfP[0]), "r"(ct.halfP[1]), "r"(ct.halfP[2]), "r"(h3), "r"(x0), "r"(x1), "r"(x2), "r"(x3));
    over = bw != 0;
  }
  uint32_t e0, e1, e2, e3;
  asm("sub.cc.u32 %0, %4, %8;\n\tsubc.cc.u32 %1, %5, %9;\n\tsubc.cc.u32 %2, %6, %10;\n\tsubc.u32 %3, %7, %11;"
      : "=r"(e0), "=r"(e1), "=r"(e2), "=r"(e3) : "r"(P0), "r"(P1), "r"(P2), "r"(P3), "r"(x0), "r"(x1), "r"(x2), "r"(x3));
  uint32_t m0 = over ? e0 : x0, m1 = over ? e1 : x1, m2 = over ? e2 : x2, m3 = over ? e3 : x3;
  int top_bit = 127 + 1022;
  if (m3 == 0u) {  // a magnitude below 2^96 (usual with 16 or 17 moduli, or after cancellation): one word up
    m3 = m2, m2 = m1, m1 = m0, m0 = 0u;
    top_bit -= 32;
  }
  const int lz = __clz(m3);
  const int e_biased = top_bit - lz - shift;  // exponent field minus one
  if (m3 == 0u || (unsigned)e_biased >= 2046u) {  // below 2^64, or a result outside the normal range: general routine
    const uint32_t mag[4] = {over ? e0 : x0, over ? e1 : x1, over ? e2 : x2, over ? e3 : x3};
    const double r = round_scaled_fast<4>(mag, shift);
    return over ? -r : r;
  }
  const uint32_t w1 = __funnelshift_l(m2, m3, lz), w0 = __funnelshift_l(m1, m2, lz);
  const uint32_t rest = __funnelshift_l(m0, m1, lz) | m0;
  uint32_t lo = __funnelshift_r(w0, w1, 11), hi = w1 >> 11;
  const uint32_t sticky = ((w0 & 0x3FFu) | rest) != 0u ? 1u : 0u;
  const uint32_t inc = (w0 >> 10) & (sticky | lo) & 1u;
  asm("add.cc.u32 %0, %0, %2;\n\taddc.u32 %1, %1, 0;" : "+r"(lo), "+r"(hi) : "r"(inc));
  hi += (uint32_t)e_biased << 20;
  if (over) hi |= 0x80000000u;
  return __hiloint2double((int)hi, (int)lo);
}

// The same for 2^128 <= P < 2^158 (20 to 24 moduli): five 64-bit column sums, x = S - q P has five words and is formed
// modulo 2^160 as acc[k] + q n_k with n = 2^160 - P.  The 32 bits of S for the quotient estimate come from bit 96 up
// (the two top column sums and the high half of the third, carries from below left out: they are worth less than
// 2^98 < P / 2^30); checked against big integers for 20 to 24 moduli.
__device__ __forceinline__ double reconstruct_lean5(const unsigned long long (&acc)[5], const CrtTable& ct, int shift) {
  uint32_t w3, t_lo, t_hi;  // S >> 96, approximately: w3 = word 3, t = words 4 and 5
  asm("add.cc.u32 %0, %3, %4;\n\t"
      "addc.cc.u32 %1, %5, %6;\n\t"
      "addc.u32 %2, %7, 0;"
      : "=r"(w3), "=r"(t_lo), "=r"(t_hi)
      : "r"((uint32_t)acc[3]), "r"((uint32_t)(acc[2] >> 32)), "r"((uint32_t)acc[4]), "r"((uint32_t)(acc[3] >> 32)), "r"((uint32_t)(acc[4] >> 32)));
  const uint32_t top = ct.q_word == 4 ? __funnelshift_r(t_lo, t_hi, ct.q_bit) : __funnelshift_r(w3, t_lo, ct.q_bit);
  const uint32_t q = __umulhi(top, ct.q_mul) >> 20;
  const uint32_t P0 = ct.P[0], P1 = ct.P[1], P2 = ct.P[2], P3 = ct.P[3], P4 = ct.P[4];
  const unsigned long long c0 = acc[0] + (unsigned long long)q * ct.negP[0];
  const unsigned long long c1 = acc[1] + (unsigned long long)q * ct.negP[1];
  const unsigned long long c2 = acc[2] + (unsigned long long)q * ct.negP[2];
  const unsigned long long c3 = acc[3] + (unsigned long long)q * ct.negP[3];
  const unsigned long long c4 = acc[4] + (unsigned long long)q * ct.negP[4];
  uint32_t x0 = (uint32_t)c0, x1, x2, x3, x4;
  asm("add.cc.u32 %0, %4, %5;\n\t"
      "addc.cc.u32 %1, %6, %7;\n\t"
      "addc.cc.u32 %2, %8, %9;\n\t"
      "addc.u32 %3, %10, %11;"
      : "=r"(x1), "=r"(x2), "=r"(x3), "=r"(x4)
      : "r"((uint32_t)(c0 >> 32)), "r"((uint32_t)c1), "r"((uint32_t)(c1 >> 32)), "r"((uint32_t)c2), "r"((uint32_t)(c2 >> 32)), "r"((uint32_t)c3),
        "r"((uint32_t)(c3 >> 32)), "r"((uint32_t)c4));
  if (x4 >= P4) {  // rarely true: x >= P needs the full comparison
    uint32_t d0, d1, d2, d3, d4, below;
    asm("sub.cc.u32 %0, %6, %11;\n\t"
        "subc.cc.u32 %1, %7, %12;\n\t"
        "subc.cc.u32 %2, %8, %13;\n\t"
        "subc.cc.u32 %3, %9, %14;\n\t"
        "subc.cc.u32 %4, %10, %15;\n\t"
        "subc.u32 %5, 0, 0;"
        : "=r"(d0), "=r"(d1), "=r"(d2), "=r"(d3), "=r"(d4), "=r"(below)
        : "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(x4), "r"(P0), "r"(P1), "r"(P2), "r"(P3), "r"(P4));
    if (!below) x0 = d0, x1 = d1, x2 = d2, x3 = d3, x4 = d4;
  }
  const uint32_t h4 = ct.halfP[4];
  bool over = x4 > h4;
  if (x4 == h4) {
    [[maybe_unused]] uint32_t u0, u1, u2, u3, u4;  // only the borrow is wanted
    uint32_t bw;
    asm("sub.cc.u32 %0, %6, %11;\n\t"
        "subc.cc.u32 %1, %7, %12;\n\t"
        "subc.cc.u32 %2, %8, %13;\n\t"
        "subc.cc.u32 %3, %9, %14;\n\t"
        "subc.cc.u32 %4, %10, %15;\n\t"
        "subc.u32 %5, 0, 0;"
        : "=r"(u0), "=r"(u1), "=r"(u2), "=r"(u3), "=r"(u4), "=r"(bw)
        : "r"(ct.halfP[0]), "r"(ct.halfP[1]), "r"(ct.halfP[2]), "r"(ct.halfP[3]), "r"(h4), "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(x4));
    over = bw != 0;
  }
  uint32_t e0, e1, e2, e3, e4;  // e = P - x
  asm("sub.cc.u32 %0, %5, %10;\n\t"
      "subc.cc.u32 %1, %6, %11;\n\t"
      "subc.cc.u32 %2, %7, %12;\n\t"
      "subc.cc.u32 %3, %8, %13;\n\t"
      "subc.u32 %4, %9, %14;"
      : "=r"(e0), "=r"(e1), "=r"(e2), "=r"(e3), "=r"(e4)
      : "r"(P0), "r"(P1), "r"(P2), "r"(P3), "r"(P4), "r"(x0), "r"(x1), "r"(x2), "r"(x3), "r"(x4));
  uint32_t m0 = over ? e0 : x0, m1 = over ? e1 : x1, m2 = over ? e2 : x2, m3 = over ? e3 : x3, m4 = over ? e4 : x4;
  int top_bit = 159 + 1022;
  if (m4 == 0u) {  // a magnitude below 2^128: one word up
    m4 = m3, m3 = m2, m2 = m1, m1 = m0, m0 = 0u;
    top_bit -= 32;
  }
  const int lz = __clz(m4);
  const int e_biased = top_bit - lz - shift;  // exponent field minus one
  if (m4 == 0u || (unsigned)e_biased >= 2046u) {  // below 2^96, or a result outside the normal range: general routine
    const uint32_t mag[5] = {over ? e0 : x0, over ? e1 : x1, over ? e2 : x2, over ? e3 : x3, over ? e4 : x4};
    const double r = round_scaled_fast<5>(mag, shift);
    return over ? -r : r;
  }
  const uint32_t w1 = __funnelshift_l(m3, m4, lz), w0 = __funnelshift_l(m2, m3, lz);
  const uint32_t rest = __funnelshift_l(m1, m2, lz) | m1 | m0;
  uint32_t lo = __funnelshift_r(w0, w1, 11), hi = w1 >> 11;
  const uint32_t sticky = ((w0 & 0x3FFu) | rest) != 0u ? 1u : 0u;
  const uint32_t inc = (w0 >> 10) & (sticky | lo) & 1u;
  asm("add.cc.u32 %0, %0, %2;\n\taddc.u32 %1, %1, 0;" : "+r"(lo), "+r"(hi) : "r"(inc));
  hi += (uint32_t)e_biased << 20;
  if (over) hi |= 0x80000000u;
  return __hiloint2double((int)hi, (int)lo);
}

// Tail shared by the reconstruction kernels: from the 64-bit column sums acc[k] = sum_l r_l w_l[k] (weight
// word k, no carries yet) to C_ij.  LEAN = 4 / 5 selects the carry-chain tails above, 0 the generic
// multiword route (any modulus count).
template <int WW, int NW, int LEAN>
__device__ __forceinline__ double finish_element(const unsigned long long (&acc)[WW], const CrtTable& ct, int shift) {
  if constexpr (LEAN == 4) {
    static_assert(LEAN != 4 || (WW == 4 && NW == 5), "this lean tail is written for 4 weight words, 5 sum words");
    unsigned long long a4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) a4[k] = acc[k < WW ? k : 0];
    return reconstruct_lean(a4, ct, shift);
  } else if constexpr (LEAN == 5) {
    static_assert(LEAN != 5 || (WW >= 5 && NW == 6), "this lean tail is written for 5 weight words, 6 sum words");
    unsigned long long a5[5];
#pragma unroll
    for (int k = 0; k < 5; ++k) a5[k] = acc[k < WW ? k : 0];
    return reconstruct_lean5(a5, ct, shift);
  } else {
    uint32_t S[NW];
    unsigned long long carry = 0ull;
#pragma unroll
    for (int k = 0; k < NW; ++k) {
      const unsigned long long v = (k < WW ? acc[k < WW ? k : 0] : 0ull) + carry;
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
    const double mag = round_scaled_fast<NW>(S, shift);
    return neg ? -mag : mag;
  }
}

// ------------------------------------------------------------------------------------
// Production kernel: the contraction S = sum_l r_l w_l (Section 5.2) runs on the tensor cores.
//
// With the weights cut into bytes, S = sum_d 2^(8d) sum_l r_l digit_d(w_l): a [rows x moduli] by
// [moduli x digits] product of bytes, every digit sum below 27 * 255 * 255 < 2^21.  A warp takes 128
// consecutive rows i of one column j (one 128-byte line of residues per modulus) and runs
// mma.sync.m16n8k32 (u8 x u8 -> s32) on them:
//   * quad g (four lanes) owns rows 16 g .. 16 g + 15; lane q of the quad loads the 16 residue bytes of the
//     moduli q, q + 4, q + 8, ... with one 16-byte load each and transposes 4 x 4 byte blocks in registers,
//     which yields its share of the A fragments (k slot 4 q + n holds modulus q + 4 n, slot 16 + 4 q + n
//     modulus q + 16 + 4 n); two rows of the quad are the MMA rows g and g + 8
//   * the B fragments are constants (host-built, CrtTable::bfrag): tiles 0 and 1 give lane q' of the quad
//     the digit sums 4 q' .. 4 q' + 3, i.e. the 64-bit column sum of weight word q'; a third tile carries the
//     digits 16 .. 23 (16 bits per lane) for more than 19 moduli
//   * the column sums of a row are then spread over the quad, so they cross once through shared memory
//     (layout below: neither the 8-byte writes nor the 16-byte reads have bank conflicts) and every lane
//     finishes four consecutive rows with the tails above.
// ------------------------------------------------------------------------------------
constexpr int kXposeQuadBytes = 16 * 32 + 4 * 16;              // 16 rows x 32 bytes, 16 bytes of padding per 4 rows
constexpr int kXposeWarpBytes = 8 * kXposeQuadBytes + 4 * 32;  // + 32 bytes per pair of quads
__host__ __device__ constexpr int kCrtWarps(int nt) { return nt == 3 ? 4 : 8; }  // warps per block: two crossing buffers per warp with three tiles
__device__ __forceinline__ uint32_t xpose_quad_offset(int g) { return (uint32_t)(g * kXposeQuadBytes + 32 * (g >> 1)); }
__device__ __forceinline__ constexpr uint32_t xpose_row_offset(int n) { return (uint32_t)(32 * n + 16 * (n >> 2)); }

__device__ __forceinline__ void mma_u8_16832(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
               : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
__device__ __forceinline__ unsigned long long mad_wide(uint32_t a, uint32_t b, uint32_t c) {  // a * b + c in 64 bits
  unsigned long long d;
  asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(d) : "r"(a), "r"(b), "l"((unsigned long long)c));
  return d;
}
__device__ __forceinline__ void sts64(uint32_t addr, unsigned long long v) {
  asm volatile("st.shared.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ void lds128(uint32_t addr, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.shared.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "r"(addr) : "memory");
}

// NT: digit tiles (2: weights of up to 128 bits, 3: up to 192); NHI: moduli beyond the 16th held per lane;
// WW / NW / LEAN as in finish_element.  The residue loads of a warp's next unit are issued before the tails of
// the current one, so their latency hides behind that arithmetic.
template <int NT, int NHI, int WW, int NW, int LEAN>
__global__ void __launch_bounds__(kCrtWarps(NT) * 32, NT == 3 ? 4 : 3)
crt_mma_kernel(const __grid_constant__ CrtTable ct, const uint8_t* __restrict__ res, size_t res_ld, size_t res_stride,
               const int32_t* __restrict__ s, const int32_t* __restrict__ t, int64_t M, int64_t N, int64_t rows_readable,
               double* __restrict__ C, int64_t ldc) {
  static_assert(WW <= 2 * NT && NT >= 2 && NT <= 3 && NHI >= 0 && NHI <= 3, "tile counts");
  constexpr int kWarps = kCrtWarps(NT);
  constexpr int NLD = 4 + NHI;  // 16-byte loads per lane and unit: moduli q, q + 4, ...
  __shared__ __align__(16) uint8_t xpose[NT == 3 ? 2 : 1][kWarps][kXposeWarpBytes];  // [1]: the third tile's sums
  constexpr uint32_t kUOffset = kWarps * kXposeWarpBytes;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, q = lane & 3;
  uint32_t bf[NT][2];
#pragma unroll
  for (int tl = 0; tl < NT; ++tl) bf[tl][0] = ct.bfrag[tl][lane][0], bf[tl][1] = ct.bfrag[tl][lane][1];
  const uint32_t xw = (uint32_t)__cvta_generic_to_shared(&xpose[0][warp][0]) + xpose_quad_offset(g);
  const uint32_t x_write = xw + 8u * q;   // + row offset: this lane's column sum for row n of the quad
  const uint32_t x_read = xw + 144u * q;  // rows 4 q .. 4 q + 3 of the quad, all four lanes' sums
  // work units (row block, column) are dealt round-robin to the warps of the grid; the position advances without
  // a division per unit
  const int64_t row_blocks = (M + 127) / 128;
  const int64_t warps_total = (int64_t)gridDim.x * kWarps;
  const int64_t step_j = warps_total / row_blocks, step_rb = warps_total - step_j * row_blocks;
  const int64_t first = (int64_t)blockIdx.x * kWarps + warp;
  int64_t j = first / row_blocks, rb = first - j * row_blocks;
  const bool vec_store = ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && ((ldc & 1) == 0);
  const int n_mine = (ct.L - q + 3) >> 2;  // this lane's moduli: q + 4 n for n < n_mine
  const uint8_t* lane_base = res + (size_t)q * res_stride + (size_t)(16 * g);
  const size_t stride4 = 4 * res_stride;
  uint32_t W[NLD][4];
  auto issue_loads = [&](int64_t jj, int64_t rr) {
    const bool readable = rr * 128 + 16 * g < rows_readable;
    const uint8_t* p = lane_base + (size_t)jj * res_ld + (size_t)(rr * 128);
#pragma unroll
    for (int n = 0; n < NLD; ++n) {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (readable && n < n_mine) v = __ldg(reinterpret_cast<const uint4*>(p));
      W[n][0] = v.x, W[n][1] = v.y, W[n][2] = v.z, W[n][3] = v.w;
      p += stride4;
    }
  };
  bool have = j < N;
  if (have) issue_loads(j, rb);
  while (have) {
    const int64_t cur_j = j, i0 = rb * 128 + 16 * g + 4 * q;  // this lane finishes rows i0 .. i0 + 3 of column cur_j
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      // 4 x 4 byte transposes: lo[r] / hi[r] = residues of row 4 c + r for this lane's moduli
      uint32_t lo[4], hi[4];
      {
        const uint32_t u0 = __byte_perm(W[0][c], W[1][c], 0x5140), u1 = __byte_perm(W[0][c], W[1][c], 0x7362);
        const uint32_t v0 = __byte_perm(W[2][c], W[3][c], 0x5140), v1 = __byte_perm(W[2][c], W[3][c], 0x7362);
        lo[0] = __byte_perm(u0, v0, 0x5410), lo[1] = __byte_perm(u0, v0, 0x7632);
        lo[2] = __byte_perm(u1, v1, 0x5410), lo[3] = __byte_perm(u1, v1, 0x7632);
      }
      if constexpr (NHI == 0) {
        hi[0] = hi[1] = hi[2] = hi[3] = 0u;
      } else if constexpr (NHI == 1) {
#pragma unroll
        for (int r = 0; r < 4; ++r) hi[r] = __byte_perm(W[NLD - 1][c], 0u, 0x4440 + r);
      } else {
        const uint32_t w5 = W[NHI >= 2 ? 5 : 0][c], w6 = NHI == 3 ? W[NHI == 3 ? 6 : 0][c] : 0u;
        const uint32_t u0 = __byte_perm(W[4][c], w5, 0x5140), u1 = __byte_perm(W[4][c], w5, 0x7362);
        const uint32_t v0 = __byte_perm(w6, 0u, 0x4140), v1 = __byte_perm(w6, 0u, 0x4342);
        hi[0] = __byte_perm(u0, v0, 0x5410), hi[1] = __byte_perm(u0, v0, 0x7632);
        hi[2] = __byte_perm(u1, v1, 0x5410), hi[3] = __byte_perm(u1, v1, 0x7632);
      }
#pragma unroll
      for (int pr = 0; pr < 2; ++pr) {
        const int ra = 4 * c + 2 * pr, rb2 = ra + 1;  // rows of the quad on MMA rows g and g + 8
        int d0[4], d1[4];
        mma_u8_16832(d0, lo[2 * pr], lo[2 * pr + 1], hi[2 * pr], hi[2 * pr + 1], bf[0][0], bf[0][1]);
        mma_u8_16832(d1, lo[2 * pr], lo[2 * pr + 1], hi[2 * pr], hi[2 * pr + 1], bf[1][0], bf[1][1]);
        // digits 4 q .. 4 q + 3 of row ra (d[0], d[1]) and of row rb2 (d[2], d[3]): sum_d 2^(8 d) D_d < 2^46
        sts64(x_write + xpose_row_offset(ra), mad_wide((uint32_t)(d1[0] + (d1[1] << 8)), 65536u, (uint32_t)(d0[0] + (d0[1] << 8))));
        sts64(x_write + xpose_row_offset(rb2), mad_wide((uint32_t)(d1[2] + (d1[3] << 8)), 65536u, (uint32_t)(d0[2] + (d0[3] << 8))));
        if constexpr (NT == 3) {
          int d2[4];
          mma_u8_16832(d2, lo[2 * pr], lo[2 * pr + 1], hi[2 * pr], hi[2 * pr + 1], bf[NT - 1][0], bf[NT - 1][1]);
          sts64(x_write + kUOffset + xpose_row_offset(ra), (unsigned long long)(uint32_t)(d2[0] + (d2[1] << 8)));
          sts64(x_write + kUOffset + xpose_row_offset(rb2), (unsigned long long)(uint32_t)(d2[2] + (d2[3] << 8)));
        }
      }
    }
    // next unit of this warp: its loads fly while the tails below run
    j += step_j, rb += step_rb;
    if (rb >= row_blocks) rb -= row_blocks, ++j;
    have = j < N;
    if (have) issue_loads(j, rb);
    __syncwarp();
    // every lane finishes its four rows two at a time (a rolled loop: the column sums are read just before use,
    // which keeps the register count low enough for three blocks per SM)
    const int tj = t[cur_j];
    double* dst = C + i0 + cur_j * ldc;
#pragma unroll 1
    for (int h = 0; h < 2; ++h) {
      double out[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const uint32_t xr = x_read + 64 * h + 32 * e;
        unsigned long long a[2 * NT];
        lds128(xr, a[0], a[1]);
        lds128(xr + 16, a[2], a[3]);
        if constexpr (NT == 3) {
          // 16-bit sums above bit 128: word 4 from lanes 0 and 1, word 5 from lanes 2 and 3
          unsigned long long u0, u1, u2, u3;
          lds128(xr + kUOffset, u0, u1);
          lds128(xr + kUOffset + 16, u2, u3);
          a[4] = u0 + (u1 << 16);
          a[5] = u2 + (u3 << 16);
        }
        const int64_t i = i0 + 2 * h + e;
        const int sh = (i < M ? s[i] : 0) + tj;
        unsigned long long aw[WW];
#pragma unroll
        for (int k = 0; k < WW; ++k) aw[k] = a[k];
        out[e] = finish_element<WW, NW, LEAN>(aw, ct, sh);
      }
      const int64_t i = i0 + 2 * h;
      if (i + 2 <= M && vec_store) {
        *reinterpret_cast<double2*>(dst + 2 * h) = make_double2(out[0], out[1]);
      } else {
        if (i < M) dst[2 * h] = out[0];
        if (i + 1 < M) dst[2 * h + 1] = out[1];
      }
    }
    __syncwarp();  // the crossing buffer is rewritten by the next unit
  }
}

__global__ void copy_residues_kernel(const uint8_t* __restrict__ res, int64_t Mp, size_t res_stride, int64_t M, int64_t N,
                                     uint8_t* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t l = blockIdx.z;
  if (i >= M) return;
  for (int64_t j = blockIdx.y; j < N; j += gridDim.y)
    out[(size_t)l * (size_t)M * (size_t)N + (size_t)j * (size_t)M + (size_t)i] =
        res[(size_t)l * res_stride + (size_t)j * (size_t)Mp + (size_t)i];
}

// acc = (acc + chunk) mod m for one modulus per blockIdx.y: sums the residues of two k ranges
// (an extension the paper does not have: it never splits K; the residue of a sum is the sum of the residues).
// 16 bytes per thread.
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
  // weight words actually used
  int ww = 1;
  for (int l = 0; l < ct.L; ++l)
    for (int k = 0; k < kCrtWords; ++k)
      if (ct.w[l][k] && k + 1 > ww) ww = k + 1;
  // The tensor-core kernel reads 16 residue bytes per load: aligned columns, and either a row count that is a
  // multiple of 16 or columns padded to one (the workspace layout).
  const int64_t rows16 = round_up(g.M, 16);
  const bool aligned = !x_out && (res_ld % 16 == 0) && (res_stride % 16 == 0) && ((reinterpret_cast<uintptr_t>(res) & 15) == 0) &&
                       res_ld >= rows16;
  if (aligned) {
    const int64_t units = ((g.M + 127) / 128) * g.N;
    // persistent grid: as many blocks as stay resident (three of eight warps, or four of four with three digit tiles)
    const int64_t wpb = ww <= 4 ? kCrtWarps(2) : kCrtWarps(3);
    const int64_t cap = (int64_t)device_sm_count() * (ww <= 4 ? 3 : 4);
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((units + wpb - 1) / wpb, cap));
    const int nhi = ct.L <= 16 ? 0 : ct.L <= 20 ? 1 : ct.L <= 24 ? 2 : 3;
    const bool lean = ct.words <= 5 && ww <= 4 && ct.p_bits >= 85 && ct.p_bits <= 126;    // 13 to 19 moduli
    const bool lean5 = ct.words <= 6 && ww <= 5 && ct.p_bits >= 129 && ct.p_bits <= 158;  // 20 to 23 moduli
#define OZK_CRT_MMA(NT, NHI, WW, NW, LEAN)                                                                           \
  crt_mma_kernel<NT, NHI, WW, NW, LEAN><<<grid, kCrtWarps(NT) * 32, 0, st>>>(ct, res, (size_t)res_ld, res_stride, s, t, g.M, g.N, rows16, C, ldc)
    bool launched = true;
    if (lean && nhi == 0) OZK_CRT_MMA(2, 0, 4, 5, 4);
    else if (lean && nhi == 1) OZK_CRT_MMA(2, 1, 4, 5, 4);
    else if (lean5 && nhi == 1) OZK_CRT_MMA(3, 1, 5, 6, 5);
    else if (lean5 && nhi == 2) OZK_CRT_MMA(3, 2, 5, 6, 5);
    else if (ww <= 4 && nhi == 0 && ct.words <= 2) OZK_CRT_MMA(2, 0, 4, 2, 0);
    else if (ww <= 4 && nhi == 0 && ct.words == 3) OZK_CRT_MMA(2, 0, 4, 3, 0);
    else if (ww <= 4 && nhi == 0 && ct.words == 4) OZK_CRT_MMA(2, 0, 4, 4, 0);
    else if (ww <= 4 && nhi == 0 && ct.words == 5) OZK_CRT_MMA(2, 0, 4, 5, 0);
    else if (ww <= 4 && nhi == 1 && ct.words == 5) OZK_CRT_MMA(2, 1, 4, 5, 0);
    else if (nhi == 1 && ct.words == 6) OZK_CRT_MMA(3, 1, 6, 6, 0);
    else if (nhi == 2 && ct.words == 6) OZK_CRT_MMA(3, 2, 6, 6, 0);
    else if (nhi == 3 && ct.words == 6) OZK_CRT_MMA(3, 3, 6, 6, 0);
    else launched = false;
#undef OZK_CRT_MMA
    if (launched) return cudaGetLastError();
  }
  dim3 grid((unsigned)((g.M + 255) / 256), (unsigned)(g.N < 65535 ? g.N : 65535));
  switch (ct.words) {
    case 2: crt_kernel<2><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc, x_out); break;
    case 3: crt_kernel<3><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc, x_out); break;
    case 4: crt_kernel<4><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc, x_out); break;
    case 5: crt_kernel<5><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc, x_out); break;
    default: crt_kernel<6><<<grid, 256, 0, st>>>(ct, res, res_ld, res_stride, s, t, g.M, g.N, C, ldc, x_out); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_copy_residues(const Geometry& g, const uint8_t* res, uint8_t* out, cudaStream_t st) {
  dim3 grid((unsigned)((g.M + 255) / 256), (unsigned)(g.N < 65535 ? g.N : 65535), (unsigned)g.L);
  copy_residues_kernel<<<grid, 256, 0, st>>>(res, g.Mp, (size_t)g.Mp * (size_t)g.Np, g.M, g.N, out);
  return cudaGetLastError();
}

}  // namespace ozk
