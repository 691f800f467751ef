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

namespace ozk {
namespace {

template <int NW>
struct Words {
  uint32_t w[NW];
};

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

__global__ void copy_residues_kernel(const uint8_t* __restrict__ res, int64_t Mp, size_t res_stride, int64_t M, int64_t N,
                                     uint8_t* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t j = blockIdx.y;
  const int64_t l = blockIdx.z;
  if (i >= M) return;
  out[(size_t)l * (size_t)M * (size_t)N + (size_t)j * (size_t)M + (size_t)i] =
      res[(size_t)l * res_stride + (size_t)j * (size_t)Mp + (size_t)i];
}

}  // namespace

cudaError_t launch_crt(const Geometry& g, const CrtTable& ct, const uint8_t* res, int64_t res_ld, size_t res_stride,
                       const int32_t* s, const int32_t* t, double* C, int64_t ldc, uint32_t* x_out, cudaStream_t st) {
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
