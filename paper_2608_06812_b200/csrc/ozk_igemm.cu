// INT8 x INT8 -> INT32 on FP4 limbs (Section 3, last paragraph; Eq. 1 with p = q = 3; Lemma 2).
//
//   encode_i8_cols / encode_i8_rows   every int8 -> three greedy base-13 limbs (|c| <= 8), one E2M1
//                                     plane per limb, K-contiguous, two nibbles per byte
//   gemm_int8 (ozk_gemm.cu)           nine limb products in five accumulators, int32 epilogue
//
// Exactness: a group holds at most three products of magnitude <= 64, so 192 K <= 2^24 keeps every
// FP32 partial sum an exact integer (K <= 87381).
#include "ozk_common.cuh"

namespace ozk {
namespace {

// Greedy decomposition (Lemma 1, Lemma 2): digit = representative of n mod 13 of smallest magnitude,
// +-5 replaced by -+8; recurse on the exact quotient.  Returns three E2M1 codes in 12 bits.
__device__ __forceinline__ uint32_t greedy_codes(int n) {
  uint32_t out = 0;
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    int r = n % 13;             // C remainder: sign of n
    if (r > 6) r -= 13;
    if (r < -6) r += 13;
    if (r == 5) r = -8;
    if (r == -5) r = 8;
    n = (n - r) / 13;           // exact
    const int a = r < 0 ? -r : r;
    // doubled magnitudes 0,1,2,3,4,6,8 -> E2M1 codes 0,1,2,3,4,5,6
    const uint32_t code = (a <= 4 ? (uint32_t)a : (a == 6 ? 5u : 6u)) | (r < 0 ? 8u : 0u);
    out |= code << (4 * i);
  }
  return out;
}

// B side: plane row = column j of B (K contiguous).  Thread = 16 consecutive k.
__global__ void __launch_bounds__(256) encode_i8_cols_kernel(const int8_t* __restrict__ B, int64_t ldb, int64_t N, int64_t K,
                                                             int64_t Kp, uint8_t* __restrict__ planes, size_t plane_bytes) {
  __shared__ uint16_t lut[256];
  lut[threadIdx.x] = (uint16_t)greedy_codes((int)threadIdx.x - 128);
  __syncthreads();
  const int64_t j = blockIdx.x;
  const int64_t k = ((int64_t)blockIdx.y * blockDim.x + threadIdx.x) * 16;
  if (k >= Kp) return;
  uint32_t w[3][2] = {{0, 0}, {0, 0}, {0, 0}};
  if (j < N) {
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      if (k + e < K) {
        const uint32_t c = lut[(int)B[j * ldb + k + e] + 128];
#pragma unroll
        for (int i = 0; i < 3; ++i) w[i][e >> 3] |= ((c >> (4 * i)) & 0xFu) << (4 * (e & 7));
      }
    }
  }
  uint8_t* dst = planes + (size_t)j * (size_t)(Kp / 2) + (size_t)(k / 2);
#pragma unroll
  for (int i = 0; i < 3; ++i) *reinterpret_cast<uint2*>(dst + (size_t)i * plane_bytes) = make_uint2(w[i][0], w[i][1]);
}

// A side: plane row = row i of A (M contiguous source).  Block = 32 rows x 64 k through shared memory.
__global__ void __launch_bounds__(256) encode_i8_rows_kernel(const int8_t* __restrict__ A, int64_t lda, int64_t M, int64_t K,
                                                             int64_t Kp, uint8_t* __restrict__ planes, size_t plane_bytes) {
  __shared__ uint16_t lut[256];
  __shared__ int8_t in_s[64][33];
  __shared__ uint32_t out_s[3][32][9];
  const int t = threadIdx.x;
  lut[t] = (uint16_t)greedy_codes(t - 128);
  const int64_t i0 = (int64_t)blockIdx.x * 32, k0 = (int64_t)blockIdx.y * 64;
  {
    const int ti = t & 31, tk = t >> 5;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      const int64_t i = i0 + ti, k = k0 + tk + 8 * n;
      in_s[tk + 8 * n][ti] = (i < M && k < K) ? A[i + k * lda] : (int8_t)0;
    }
  }
  __syncthreads();
  const int r = t & 31, g = t >> 5;
  uint32_t w[3] = {0, 0, 0};
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const uint32_t c = lut[(int)in_s[8 * g + e][r] + 128];
#pragma unroll
    for (int i = 0; i < 3; ++i) w[i] |= ((c >> (4 * i)) & 0xFu) << (4 * e);
  }
#pragma unroll
  for (int i = 0; i < 3; ++i) out_s[i][r][g] = w[i];
  __syncthreads();
  const int row = t >> 3, word = t & 7;
  uint8_t* dst = planes + (size_t)(i0 + row) * (size_t)(Kp / 2) + (size_t)(k0 / 2) + 4 * word;
#pragma unroll
  for (int i = 0; i < 3; ++i) *reinterpret_cast<uint32_t*>(dst + (size_t)i * plane_bytes) = out_s[i][row][word];
}

struct I8Geometry {
  int64_t Mp, Np, Kp;
  size_t off_planes_a, off_planes_b, total;
};

bool make_i8_geometry(int64_t M, int64_t N, int64_t K, I8Geometry* g) {
  if (M < 0 || N < 0 || K < 0) return false;
  g->Mp = round_up(M > 0 ? M : 1, kTileRows);
  g->Np = round_up(N > 0 ? N : 1, kTileRows);
  g->Kp = round_up(K > 0 ? K : 1, kTileKNibbles);
  size_t off = 1024;  // status block
  g->off_planes_a = off;
  off += 3 * (size_t)g->Mp * (size_t)(g->Kp / 2);
  g->off_planes_b = off;
  off += 3 * (size_t)g->Np * (size_t)(g->Kp / 2);
  g->total = (off + 1023) / 1024 * 1024;
  return true;
}

}  // namespace
}  // namespace ozk

using namespace ozk;

extern "C" {

size_t ozk_igemm_i8_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  I8Geometry g;
  return make_i8_geometry(M, N, K, &g) ? g.total : 0;
}

ozk_status ozk_igemm_i8(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda, const int8_t* B, int64_t ldb,
                        int32_t* C, int64_t ldc, void* stream) {
  I8Geometry g;
  if (!make_i8_geometry(M, N, K, &g)) return OZK_ERR_INVALID_ARG;
  if (K > 87381) return OZK_ERR_UNSUPPORTED;  // 3 * 64 * K <= 2^24 (Lemma 2 with n_g = 3)
  if (N > 65535 * 128ll || g.Mp / 32 > 65535 * 32ll) return OZK_ERR_UNSUPPORTED;
  uint8_t* ws = workspace_ptr();
  if (!ws || workspace_bytes() < g.total) return OZK_ERR_WORKSPACE;
  if (M == 0 || N == 0) return OZK_OK;
  if (!C || ldc < M || (K > 0 && (!A || !B)) || lda < (M > 1 ? M : 1) || ldb < (K > 1 ? K : 1)) return OZK_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return OZK_ERR_CUDA;
  if (major != 10) return OZK_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t pa = (size_t)g.Mp * (size_t)(g.Kp / 2), pb = (size_t)g.Np * (size_t)(g.Kp / 2);
  {
    dim3 grid((unsigned)(g.Mp / 32), (unsigned)(g.Kp / 64));
    encode_i8_rows_kernel<<<grid, 256, 0, st>>>(A, lda, M, K, g.Kp, ws + g.off_planes_a, pa);
  }
  {
    dim3 grid((unsigned)g.Np, (unsigned)((g.Kp + 4095) / 4096));
    encode_i8_cols_kernel<<<grid, 256, 0, st>>>(B, ldb, N, K, g.Kp, ws + g.off_planes_b, pb);
  }
  if (cudaGetLastError() != cudaSuccess) return OZK_ERR_CUDA;
  return gemm_int8(ws + g.off_planes_a, ws + g.off_planes_b, M, N, g.Mp, g.Np, g.Kp, C, ldc, reinterpret_cast<StatusBlock*>(ws), st);
}

}  // extern "C"
