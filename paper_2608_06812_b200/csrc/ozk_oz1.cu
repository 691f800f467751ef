// Ozaki scheme I on base-13 E2M1 limbs (Section 4): p = q = 15 greedy limbs per converted integer,
// limb products aggregated along anti-diagonals i + j = g and weighted by 13^g (Eq. 1, Fig. 2).
//
//   stage 1  shared-exponent conversion with c = 53 (Section 4.2), then the / 13 recursion of Lemma 1
//            writes 15 limb planes per operand in one sweep (Section 6.2)
//   stage 2  the 15 x 15 limb products run as 20 passes of 4 x 3 limbs on the tensor cores; a pass
//            keeps its six anti-diagonals in tensor memory and stores one int64 block value per
//            output element (ozk_gemm.cu)
//   stage 3  one reduction kernel: X = sum_passes 13^(4 bp + 3 bq) V_pass in multiword integers,
//            then inverse scaling and one rounding to FP64 (Section 4.2)
//
// Exactness (Lemma 2 for a 4 x 3 block): at most three products of magnitude <= 64 share an FP32
// accumulator, so 192 K <= 2^24, K <= 87381.
#include <string.h>

#include "ozk_common.cuh"
#include "ozk_convert.cuh"
#include "ozk_round.cuh"

namespace ozk {
namespace {

constexpr int kLimbs = 15;
constexpr int kPassW = 80;      // column-side tile width of a pass
constexpr int kPasses = 20;     // 4 row-side groups x 5 column-side groups
constexpr uint32_t kPow5 = 371293u;  // 13^5

// One greedy digit (Lemma 1, Lemma 2): representative of v mod 13 of smallest magnitude, +-5 -> -+8.
// Updates v to the exact quotient (v - c) / 13 and returns the E2M1 code of c / 2.
__device__ __forceinline__ uint32_t greedy_step(uint32_t& v) {
  const uint32_t r = v % 13u;
  int c = r > 6u ? (int)r - 13 : (int)r;
  if (c == 5) c = -8;
  if (c == -5) c = 8;
  v = (uint32_t)((int)v - c) / 13u;
  const int a = c < 0 ? -c : c;
  return (a <= 4 ? (uint32_t)a : (a == 6 ? 5u : 6u)) | (c < 0 ? 8u : 0u);
}

// Fifteen greedy limbs of a magnitude <= 2^53 < X_15, as E2M1 codes; `flip` = 8 negates every limb
// (the greedy decomposition of -n is the negated decomposition of n: S is symmetric).
__device__ __forceinline__ void decompose15(unsigned long long mag, uint32_t flip, uint32_t (&codes)[kLimbs]) {
  // mag = h2 * 13^10 + h1 * 13^5 + h0: three 32-bit pieces, the carry of one piece joins the next
  const unsigned long long n1 = mag / kPow5;
  uint32_t v = (uint32_t)(mag - n1 * kPow5);
  const unsigned long long n2 = n1 / kPow5;
  const uint32_t h1 = (uint32_t)(n1 - n2 * kPow5), h2 = (uint32_t)n2;
#pragma unroll
  for (int d = 0; d < 5; ++d) codes[d] = greedy_step(v);
  v += h1;
#pragma unroll
  for (int d = 5; d < 10; ++d) codes[d] = greedy_step(v);
  v += h2;
#pragma unroll
  for (int d = 10; d < 15; ++d) codes[d] = greedy_step(v);
#pragma unroll
  for (int d = 0; d < kLimbs; ++d) codes[d] ^= (codes[d] & 7u) ? flip : 0u;  // no negative zeros
}

// B side: plane row = column j of B (K contiguous).  Thread = 8 consecutive k, 16 planes written
// (plane 15 is the all-zero pad that completes the fourth row-side group).
__global__ void __launch_bounds__(256) oz1_encode_cols_kernel(const double* __restrict__ B, int64_t ldb, int64_t N, int64_t K,
                                                              int64_t Kp, const int32_t* __restrict__ shifts,
                                                              uint8_t* __restrict__ planes, size_t plane_bytes) {
  const int64_t j = blockIdx.x;
  const int64_t k = ((int64_t)blockIdx.y * blockDim.x + threadIdx.x) * 8;
  if (k >= Kp) return;
  uint32_t w[kLimbs];
#pragma unroll
  for (int d = 0; d < kLimbs; ++d) w[d] = 0;
  if (j < N && k < K) {
    const int s = shifts[j];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (k + e < K) {
        bool neg;
        const unsigned long long mag = to_integer_magnitude(__ldg(B + j * ldb + k + e), s, &neg);
        uint32_t codes[kLimbs];
        decompose15(mag, neg ? 8u : 0u, codes);
#pragma unroll
        for (int d = 0; d < kLimbs; ++d) w[d] |= codes[d] << (4 * e);
      }
    }
  }
  uint8_t* dst = planes + (size_t)j * (size_t)(Kp / 2) + (size_t)(k / 2);
#pragma unroll
  for (int d = 0; d < kLimbs; ++d) *reinterpret_cast<uint32_t*>(dst + (size_t)d * plane_bytes) = w[d];
  *reinterpret_cast<uint32_t*>(dst + (size_t)kLimbs * plane_bytes) = 0u;
}

// A side: plane row = row i of A (M contiguous source): 32 x 64 tile through shared memory, like the
// scheme-II encoder.
__global__ void __launch_bounds__(256) oz1_encode_rows_kernel(const double* __restrict__ A, int64_t lda, int64_t M, int64_t K,
                                                              int64_t Kp, const int32_t* __restrict__ shifts,
                                                              uint8_t* __restrict__ planes, size_t plane_bytes) {
  __shared__ double in_s[64 * 32];
  __shared__ uint32_t out_s[kLimbs][32][9];
  const int t = threadIdx.x;
  const int64_t i0 = (int64_t)blockIdx.x * 32, k0 = (int64_t)blockIdx.y * 64;
  {
    const int ti = t & 31, tk = t >> 5;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      const int64_t i = i0 + ti, k = k0 + tk + 8 * n;
      in_s[(tk + 8 * n) * 32 + ti] = (i < M && k < K) ? __ldg(A + i + k * lda) : 0.0;
    }
  }
  __syncthreads();
  const int r = t & 31, g = t >> 5;
  uint32_t w[kLimbs];
#pragma unroll
  for (int d = 0; d < kLimbs; ++d) w[d] = 0;
  const int s = shifts[i0 + r];  // Mp entries, 0 in the padding
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    bool neg;
    const unsigned long long mag = to_integer_magnitude(in_s[(8 * g + e) * 32 + r], s, &neg);
    uint32_t codes[kLimbs];
    decompose15(mag, neg ? 8u : 0u, codes);
#pragma unroll
    for (int d = 0; d < kLimbs; ++d) w[d] |= codes[d] << (4 * e);
  }
#pragma unroll
  for (int d = 0; d < kLimbs; ++d) out_s[d][r][g] = w[d];
  __syncthreads();
  const int row = t >> 3, word = t & 7;
  uint8_t* dst = planes + (size_t)(i0 + row) * (size_t)(Kp / 2) + (size_t)(k0 / 2) + 4 * word;
#pragma unroll
  for (int d = 0; d < kLimbs; ++d) *reinterpret_cast<uint32_t*>(dst + (size_t)d * plane_bytes) = out_s[d][row][word];
}

// Powers of 13 as three 32-bit words: 13^24 < 2^89.
struct Pow13Table {
  uint32_t w[25][3];
};

// Reduction (Fig. 2: "x 13^g"): X = sum over the 20 passes of 13^(4 bp + 3 bq) V, in 192-bit integers with
// separate sums for positive and negative block values; then 2^-(s_i + t_j) and one rounding.
__global__ void __launch_bounds__(256) oz1_reduce_kernel(const __grid_constant__ Pow13Table pw, const long long* __restrict__ vals,
                                                         int64_t ld, size_t pass_stride, const int32_t* __restrict__ s,
                                                         const int32_t* __restrict__ t, int64_t M, int64_t N,
                                                         double* __restrict__ C, int64_t ldc) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  for (int64_t j = blockIdx.y; j < N; j += gridDim.y) {
    const long long* vp = vals + (size_t)j * (size_t)ld + (size_t)i;
    long long v[kPasses];
#pragma unroll
    for (int l = 0; l < kPasses; ++l) v[l] = __ldg(vp + (size_t)l * pass_stride);
    uint32_t pos[6] = {0, 0, 0, 0, 0, 0}, neg[6] = {0, 0, 0, 0, 0, 0};
#pragma unroll
    for (int l = 0; l < kPasses; ++l) {
      const int e = 4 * (l / 5) + 3 * (l % 5);  // power of 13 of the block's first product
      const bool is_neg = v[l] < 0;
      const unsigned long long a = is_neg ? (unsigned long long)(-v[l]) : (unsigned long long)v[l];
      const uint32_t a0 = (uint32_t)a, a1 = (uint32_t)(a >> 32);
      // prod = a * 13^e (at most 41 + 89 bits): a0 * w into words 0..3, a1 * w into words 1..4
      uint32_t prod[6] = {0, 0, 0, 0, 0, 0}, high[6] = {0, 0, 0, 0, 0, 0};
      unsigned long long c0 = 0, c1 = 0;
#pragma unroll
      for (int k = 0; k < 3; ++k) {
        c0 += (unsigned long long)a0 * pw.w[e][k];
        prod[k] = (uint32_t)c0;
        c0 >>= 32;
        c1 += (unsigned long long)a1 * pw.w[e][k];
        high[k + 1] = (uint32_t)c1;
        c1 >>= 32;
      }
      prod[3] = (uint32_t)c0;
      high[4] = (uint32_t)c1;
      add_in_place<6>(prod, high);
      if (is_neg)
        add_in_place<6>(neg, prod);
      else
        add_in_place<6>(pos, prod);
    }
    const bool negative = !ge<6>(pos, neg);
    uint32_t mag[6];
#pragma unroll
    for (int k = 0; k < 6; ++k) mag[k] = negative ? neg[k] : pos[k];
    sub_in_place<6>(mag, negative ? pos : neg);
    const double r = round_scaled<6>(mag, s[i] + t[j]);
    C[i + j * ldc] = negative ? -r : r;
  }
}

struct Oz1Geometry {
  Geometry g;           // the part shared with the scheme-II scan (status, amax, s, t)
  size_t off_planes_a, off_planes_b, off_vals;
  size_t plane_a, plane_b;
  int64_t vals_ld;
  size_t total;
};

bool make_oz1_geometry(int64_t M, int64_t N, int64_t K, Oz1Geometry* o) {
  if (M < 0 || N < 0 || K < 0) return false;
  Geometry& g = o->g;
  memset(&g, 0, sizeof g);
  g.M = M, g.N = N, g.K = K, g.L = 0;
  g.Mp = round_up(M > 0 ? M : 1, kTileRows);
  g.Np = round_up(N > 0 ? N : 1, kTileRows);
  g.Kp = round_up(K > 0 ? K : 1, kTileKNibbles);
  g.c_bits = 53;  // c = floor(log2 min(X_15, 2^53)) (Section 4.2)
  auto up = [](size_t x) { return (x + 1023) / 1024 * 1024; };
  size_t off = 0;
  g.off_status = off;
  off += 1024;
  g.off_amax_a = off;
  off += (size_t)g.Mp * 8;
  g.off_amax_b = off;
  off += (size_t)g.Np * 8;
  off = up(off);
  g.off_s = off;
  off += up((size_t)g.Mp * 4);
  g.off_t = off;
  off += up((size_t)g.Np * 4);
  o->plane_a = (size_t)g.Mp * (size_t)(g.Kp / 2);
  o->plane_b = (size_t)g.Np * (size_t)(g.Kp / 2);
  o->off_planes_a = off;
  off += kLimbs * o->plane_a;
  o->off_planes_b = off;
  off += (kLimbs + 1) * o->plane_b;
  o->vals_ld = (int64_t)((M + kPassW - 1) / kPassW) * kPassW;
  if (o->vals_ld == 0) o->vals_ld = kPassW;
  o->off_vals = off;
  off += (size_t)kPasses * (size_t)g.Np * (size_t)o->vals_ld * sizeof(long long);
  o->total = up(off);
  g.total = o->total;
  return true;
}

void build_pow13(Pow13Table* t) {
  unsigned __int128 v = 1;
  for (int e = 0; e < 25; ++e) {
    t->w[e][0] = (uint32_t)v;
    t->w[e][1] = (uint32_t)(v >> 32);
    t->w[e][2] = (uint32_t)(v >> 64);
    v *= 13;
  }
}

}  // namespace
}  // namespace ozk

using namespace ozk;

extern "C" {

size_t ozk_dgemm_oz1_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  Oz1Geometry o;
  return make_oz1_geometry(M, N, K, &o) ? o.total : 0;
}

ozk_status ozk_dgemm_oz1(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb,
                         double* C, int64_t ldc, void* stream) {
  Oz1Geometry o;
  if (!make_oz1_geometry(M, N, K, &o)) return OZK_ERR_INVALID_ARG;
  if (K > 87381) return OZK_ERR_UNSUPPORTED;  // 3 * 64 * K <= 2^24 per accumulator of a 4 x 3 block
  if (N > 65535 * 64ll || o.g.Mp / 32 > 65535) return OZK_ERR_UNSUPPORTED;
  uint8_t* ws = workspace_ptr();
  if (!ws || workspace_bytes() < o.total) return OZK_ERR_WORKSPACE;
  if (M == 0 || N == 0) return OZK_OK;
  if (!C || ldc < M || (K > 0 && (!A || !B)) || lda < (M > 1 ? M : 1) || ldb < (K > 1 ? K : 1)) return OZK_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return OZK_ERR_CUDA;
  if (major != 10) return OZK_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Geometry& g = o.g;
  if (launch_scan_and_shifts(g, A, lda, B, ldb, ws, st) != cudaSuccess) return OZK_ERR_CUDA;
  const int32_t* s = reinterpret_cast<const int32_t*>(ws + g.off_s);
  const int32_t* t = reinterpret_cast<const int32_t*>(ws + g.off_t);
  {
    dim3 grid((unsigned)(g.Mp / 32), (unsigned)(g.Kp / 64));
    oz1_encode_rows_kernel<<<grid, 256, 0, st>>>(A, lda, M, K, g.Kp, s, ws + o.off_planes_a, o.plane_a);
  }
  {
    dim3 grid((unsigned)g.Np, (unsigned)((g.Kp + 2047) / 2048));
    oz1_encode_cols_kernel<<<grid, 256, 0, st>>>(B, ldb, N, K, g.Kp, t, ws + o.off_planes_b, o.plane_b);
  }
  if (cudaGetLastError() != cudaSuccess) return OZK_ERR_CUDA;
  long long* vals = reinterpret_cast<long long*>(ws + o.off_vals);
  ozk_status rc = gemm_oz1_passes(ws + o.off_planes_a, ws + o.off_planes_b, g.Mp, g.Np, g.Kp, M, vals, o.vals_ld,
                                  reinterpret_cast<StatusBlock*>(ws + g.off_status), st);
  if (rc != OZK_OK) return rc;
  Pow13Table pw;
  build_pow13(&pw);
  dim3 grid((unsigned)((M + 255) / 256), (unsigned)(N < 65535 ? N : 65535));
  oz1_reduce_kernel<<<grid, 256, 0, st>>>(pw, vals, o.vals_ld, (size_t)g.Np * (size_t)o.vals_ld, s, t, M, N, C, ldc);
  return cudaGetLastError() == cudaSuccess ? OZK_OK : OZK_ERR_CUDA;
}

}  // extern "C"
