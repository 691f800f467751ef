// Multiword helpers shared by the reconstruction kernels: comparisons and in-place add / subtract on
// little-endian 32-bit words, and the single rounding of (magnitude * 2^-shift) to FP64 (Section 4.2:
// the integer result is scaled back by 2^-(s_i + t_j) and rounded once, ties to even).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ozk {

template <int NW>
__device__ __forceinline__ bool ge(const uint32_t (&a)[NW], const uint32_t* b) {  // a >= b
#pragma unroll
  for (int i = NW - 1; i >= 0; --i) {
    if (a[i] != b[i]) return a[i] > b[i];
  }
  return true;
}
template <int NW>
__device__ __forceinline__ bool gt(const uint32_t (&a)[NW], const uint32_t* b) {  // a > b
#pragma unroll
  for (int i = NW - 1; i >= 0; --i) {
    if (a[i] != b[i]) return a[i] > b[i];
  }
  return false;
}
template <int NW>
__device__ __forceinline__ void sub_in_place(uint32_t (&a)[NW], const uint32_t* b) {  // a -= b (mod 2^(32 NW))
  uint32_t borrow = 0;
#pragma unroll
  for (int i = 0; i < NW; ++i) {
    const uint64_t t = (uint64_t)a[i] - b[i] - borrow;
    a[i] = (uint32_t)t;
    borrow = (uint32_t)(t >> 63);
  }
}
template <int NW>
__device__ __forceinline__ void add_in_place(uint32_t (&a)[NW], const uint32_t* b) {
  uint32_t carry = 0;
#pragma unroll
  for (int i = 0; i < NW; ++i) {
    const uint64_t t = (uint64_t)a[i] + b[i] + carry;
    a[i] = (uint32_t)t;
    carry = (uint32_t)(t >> 32);
  }
}

// RN_even(mag * 2^-shift) for a multiword magnitude; subnormal results are rounded once too.
template <int NW>
__device__ __forceinline__ double round_scaled(const uint32_t (&mag)[NW], int shift) {
  int top = -1;
#pragma unroll
  for (int i = 0; i < NW; ++i)
    if (mag[i]) top = i;
  if (top < 0) return 0.0;
  uint32_t topw = 0;
#pragma unroll
  for (int i = 0; i < NW; ++i)
    if (i == top) topw = mag[i];
  const int bitlen = 32 * top + 32 - __clz(topw);
  const int e_out = bitlen - 1 - shift;  // value in [2^e_out, 2^(e_out+1))
  int keep = 53;
  if (e_out < -1022) keep = e_out + 1075;  // bits above the subnormal grid 2^-1074
  if (keep < 0) return 0.0;               // below half of the smallest subnormal
  const int drop = bitlen - keep;
  unsigned long long q;
  int le;  // exponent of q's last bit
  if (drop <= 0) {
    q = (unsigned long long)mag[0] | (NW > 1 ? (unsigned long long)mag[1] << 32 : 0ull);
    le = -shift;
  } else {
    const int wi = drop >> 5, bi = drop & 31;
    uint32_t w0 = 0, w1 = 0, w2 = 0;
#pragma unroll
    for (int i = 0; i < NW; ++i) {
      if (i == wi) w0 = mag[i];
      if (i == wi + 1) w1 = mag[i];
      if (i == wi + 2) w2 = mag[i];
    }
    q = (((unsigned long long)w1 << 32) | w0) >> bi;
    if (bi) q |= (unsigned long long)w2 << (64 - bi);
    if (keep < 64) q &= (keep == 0) ? 0ull : ((~0ull) >> (64 - keep));
    const int rb = drop - 1;  // position of the round bit
    uint32_t round_bit = 0, sticky = 0;
#pragma unroll
    for (int i = 0; i < NW; ++i) {
      const int below = rb - 32 * i;  // how many bits of word i lie below the round bit
      if (below >= 32) {
        sticky |= mag[i];
      } else if (below >= 0) {
        sticky |= mag[i] & ((1u << below) - 1u);
        round_bit = (mag[i] >> below) & 1u;
      }
    }
    if (round_bit && (sticky || (q & 1ull))) ++q;
    le = drop - shift;
  }
  double r = (double)q;  // q <= 2^53: exact
  // exact scaling by 2^le in up to three steps, each factor a normal power of two
#pragma unroll
  for (int step = 0; step < 3; ++step) {
    const int e = max(-1000, min(1000, le));
    r *= __longlong_as_double((long long)(e + 1023) << 52);
    le -= e;
  }
  return r;
}

}  // namespace ozk
